// Sparse flash attention on the 5th-generation tensor cores (sm_100a): bf16 inputs, head_dim 128 or 64.
//
// One persistent CTA per SM walks the work list of the mask blob.  A work item is a pair of adjacent
// 128-row query blocks (2p, 2p+1) of one (sequence, head): two query tiles ("streams" A and B) share every
// K / V tile that either of them lists, so a kv tile is brought into shared memory once per 256 query rows.
// Warp roles:
//   warp 0      TMA producer: both Q tiles once per item, then K and V of every kv tile in the union of
//               the two tile lists ("step") into a ring of 32 KB shared-memory slots (128-byte swizzle); for
//               every step it leaves a descriptor word in shared memory (which streams have a tile in it, whether
//               it is a stream's last, whether the item goes on), and for every item a record for the softmax
//               warps (item, first tile entries, the head's bit-set pointers);
//   warp 1      MMA issuer (one elected thread), driven by those descriptors alone (it reads no global memory):
//               S_X = Q_X K^T into the stream's TMEM columns, then O_X += P_X V with P_X read from TMEM (it
//               overwrites the first half of S_X); the two streams are interleaved so that one stream's softmax
//               runs under the other stream's MMAs;
//   warps 2-3   idle: they fill the first warpgroup, which gives most of its registers to the other two;
//   warps 4-7   softmax of stream A, warps 8-11 of stream B: one thread per query row reads its S row from
//               TMEM (twice: running max, then probabilities), applies the tile's mask bits where the tile
//               is not fully active, writes P (bf16) back to TMEM, rescales O in TMEM when the running max
//               moved by more than 2^8, and finally normalises and stores O and the log-sum-exp.
// Only the tiles the mask lists are ever loaded or multiplied (paper Sec. 4.3: masked logits are -inf).
// Every wait is bounded; an expired wait sets the status word in the scratch buffer and the CTA drains
// and exits.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "dam_internal.cuh"
#include "sm100_ptx.cuh"

using namespace sm100;

namespace {

constexpr int kSlots = 4;
constexpr int kStageBytes = 16384;   // per-stream staging of one 64-column half of the O tile
constexpr int kSlotBytes = 32768;
constexpr int kThreads = 384;   // three warpgroups: {producer, MMA issuer, two idle warps}, softmax of stream A, softmax of stream B
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;      // S_A at 0, S_B at 128 (P_X overwrites columns [0, 64) of S_X)
constexpr uint32_t kColO = 256;    // O_A at 256, O_B at 384
constexpr float kRescaleThreshold = 8.0f;
constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr int kSchedNoSteps = 1 << 30;       // work-list entry handed to the consumers: nothing to multiply for it
// Step descriptor bits: stream A / B has a tile in the step; it is the stream's last tile of the item; the item has
// another step.
constexpr uint32_t kStepA = 1u, kStepB = 2u, kStepLastA = 4u, kStepLastB = 8u, kStepMore = 16u;
constexpr int kPolyPer8 = 2;   // of every 8 exponentials, how many use the FMA-pipe polynomial (0, 2 or 4)

struct SmemLayout {
  static constexpr int q = 0;                           // Q_A, Q_B
  static constexpr int slots = 2 * kSlotBytes;
  static constexpr int stage = kSlotBytes * (2 + kSlots);           // two staging buffers (stream A, B)
  static constexpr int bars = stage + 2 * kStageBytes;
  // q_full, q_empty, slot_full[kSlots], slot_empty[kSlots], s_full[2], p_full[2], o_final[2],
  // sched_full[2], sched_empty[2]
  static constexpr int n_bars = 2 + 2 * kSlots + 10;
  static constexpr int sched_items = bars + 8 * n_bars;     // int[2]: work-list positions handed to the consumers
  static constexpr int step_desc = sched_items + 8;         // u32[16]: what the producer found at each step (kStep*)
  static constexpr int item_rec = (step_desc + 64 + 15) & ~15;   // ItemRec[2] (16-byte aligned): what the softmax warps need to start an item
  static constexpr int tmem_slot = item_rec + 2 * 96;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int total = abort_flag + 4;
};
static_assert(SmemLayout::item_rec % 16 == 0 && SmemLayout::bars % 8 == 0, "shared-memory records must be aligned");
constexpr int kSmemBytes = SmemLayout::total + 1024;   // + slack for the 1024-byte alignment

// What the producer hands to the softmax warps with every work-list position: the item record, the first tile
// entry of each stream and the head's bit-set pointers, so that their set-up reads shared memory instead of
// walking item -> sequence record -> tile list in global memory.
struct ItemRec {
  uint4 u, v;               // the two words of the DamItem
  uint32_t eA, eB, pad0, pad1;
  DamHeadBits hb;
};
static_assert(sizeof(ItemRec) == 96, "ItemRec must be 96 bytes");

struct AttnParams {
  const unsigned char* blob;
  __nv_bfloat16* O;
  float* lse;
  uint32_t* status;         // scratch status word
  uint32_t* work_counter;   // scratch word 2, zero at launch
  unsigned long long scratch_bytes;
  int Hq, group, total_tokens, causal;
  int64_t o_stride_tok, o_stride_head;
  float scale_log2;         // softmax scale * log2(e)
  const int32_t* ranges;    // row ranges [begin, end) per sequence (chunked prefill), or NULL
};

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One work item: a pair of query blocks of one (sequence, head) and the tile-list ranges of both.
struct Item {
  int head, tok0, qb0, S, hasB, seq;
  uint32_t a0, a1, b0, b1;      // tile list [a0, a1) of block 2p, [b0, b1) of block 2p+1
};

__device__ __forceinline__ Item item_from_words(const uint4& u, const uint4& v) {
  Item it;
  it.head = (int)u.x; it.tok0 = (int)u.y; it.qb0 = (int)u.z; it.S = (int)u.w;
  it.a0 = v.x; it.a1 = v.y; it.b0 = v.y; it.b1 = v.z;
  it.hasB = (int)(v.w >> 31); it.seq = (int)(v.w & 0x7FFFFFFFu);
  return it;
}

// Merge of the two ascending tile lists: every step is one kv tile with the kinds it has in A and in B.
struct Walker {
  const uint32_t* tiles;
  uint32_t ia, ea, ib, eb, ca, cb;
  __device__ __forceinline__ void init(const uint32_t* t, const Item& it) {
    tiles = t; ia = it.a0; ea = it.a1; ib = it.b0; eb = it.b1;
    ca = ia < ea ? __ldg(tiles + ia) : kNone;
    cb = ib < eb ? __ldg(tiles + ib) : kNone;
  }
  // Order inside a row list: gathered-column tiles first (ascending index), then kv tiles (ascending).
  static __device__ __forceinline__ uint32_t key(uint32_t e) {
    if (e == kNone) return kNone;
    return (e >> 28) == DAM_KIND_GATHERED ? (e & 0xFFFFu) : ((e & 0x0FFFFFFFu) | 0x10000000u);
  }
  // One step: kb = kv tile index, or gathered tile index when the kinds are DAM_KIND_GATHERED.
  __device__ __forceinline__ bool next(int& kb, uint32_t& kindA, uint32_t& kindB) {
    const uint32_t ja = key(ca), jb = key(cb);
    const uint32_t k = ja < jb ? ja : jb;
    if (k == kNone) return false;
    kb = (int)(k & 0x0FFFFFFFu);
    kindA = (ja == k) ? (ca >> 28) : 0u;
    kindB = (jb == k) ? (cb >> 28) : 0u;
    if (ja == k) { ++ia; ca = ia < ea ? __ldg(tiles + ia) : kNone; }
    if (jb == k) { ++ib; cb = ib < eb ? __ldg(tiles + ib) : kNone; }
    return true;
  }
  __device__ __forceinline__ bool a_done() const { return ia >= ea; }
  __device__ __forceinline__ bool b_done() const { return ib >= eb; }
};

__device__ __forceinline__ uint32_t pick_word(const uint4& b, int c) {
  return c == 0 ? b.x : (c == 1 ? b.y : (c == 2 ? b.z : b.w));
}


// ---- packed fp32x2 arithmetic (one instruction for two lanes of a register pair) -----------------------
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
      "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

// 2^y for a pair of values on the FMA / ALU pipes instead of the special-function unit: split y into its
// nearest integer (added to the exponent field) and a remainder in [-0.5, 0.5] (degree-3 minimax polynomial,
// relative error 7.6e-5, far below the bf16 rounding of P).  y is clamped at -125 so that the exponent stays
// in range; that turns an underflowing probability into 2^-125 instead of 0.
__device__ __forceinline__ void ex2_poly2(float y0, float y1, float& p0, float& p1) {
  const float kMagic = 12582912.f;    // 1.5 * 2^23: adding it leaves round(y) in the low mantissa bits
  y0 = fmaxf(y0, -125.f); y1 = fmaxf(y1, -125.f);
  float r0, r1, i0, i1, f0, f1, q0, q1;
  add2(r0, r1, y0, y1, kMagic, kMagic);
  add2(i0, i1, r0, r1, -kMagic, -kMagic);
  add2(f0, f1, y0, y1, -i0, -i1);
  fma2(q0, q1, f0, f1, 0.05520550534129143f, 0.05520550534129143f, 0.24261397123336792f, 0.24261397123336792f);
  fma2(q0, q1, q0, q1, f0, f1, 0.6932547688484192f, 0.6932547688484192f);
  fma2(q0, q1, q0, q1, f0, f1, 0.9999276995658875f, 0.9999276995658875f);
  p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(r0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(r1) << 23));
}

// Sweep 1 over one S row held in TMEM (4 chunks of 32 columns, next chunk in flight while one is reduced).
template <bool MASKED>
__device__ __forceinline__ float sweep_max(uint32_t tS, const uint4& bits) {
  uint32_t ra[32], rb[32];
  float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
  tmem_ld32(tS, ra);
  tc_wait_ld();
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t* cur = (c & 1) ? rb : ra;
    uint32_t* nxt = (c & 1) ? ra : rb;
    if (c < 3) tmem_ld32(tS + (c + 1) * 32, nxt);
    const uint32_t word = pick_word(bits, c);
#pragma unroll
    for (int q = 0; q < 32; q += 4) {
      float v0 = __uint_as_float(cur[q]), v1 = __uint_as_float(cur[q + 1]);
      float v2 = __uint_as_float(cur[q + 2]), v3 = __uint_as_float(cur[q + 3]);
      if (MASKED) {
        v0 = ((word >> q) & 1u) ? v0 : -CUDART_INF_F;
        v1 = ((word >> (q + 1)) & 1u) ? v1 : -CUDART_INF_F;
        v2 = ((word >> (q + 2)) & 1u) ? v2 : -CUDART_INF_F;
        v3 = ((word >> (q + 3)) & 1u) ? v3 : -CUDART_INF_F;
      }
      mx0 = max3(mx0, v0, v1); mx1 = max3(mx1, v2, v3);
    }
    if (c < 3) tc_wait_ld();
  }
  return fmaxf(mx0, mx1);
}

// Sweep 2: p = 2^(s * scale + neg_m) for the row, packed to bf16 and stored over the first 64 columns of the
// row's S (chunk c+1 is in registers before chunk c's columns are overwritten).  Of every 8 probabilities, 6
// go through the special-function unit and 2 through the polynomial.  Returns the row sum (fp32, before the
// bf16 rounding).  A masked tile skips the arithmetic of a 32-column chunk that is inactive for every row of
// the warp.
template <bool MASKED>
__device__ __forceinline__ void exp_chunk(const uint32_t* cur, uint32_t word, float scale, float neg_m, uint32_t* pk,
                                          float& s0, float& s1, float& s2, float& s3) {
  const bool live = !MASKED || __any_sync(0xFFFFFFFFu, word != 0u);
  if (live) {
#pragma unroll
    for (int q = 0; q < 32; q += 8) {
      float y[8], p[8];
#pragma unroll
      for (int u = 0; u < 8; u += 2)
        fma2(y[u], y[u + 1], __uint_as_float(cur[q + u]), __uint_as_float(cur[q + u + 1]), scale, scale, neg_m, neg_m);
#pragma unroll
      for (int u = 0; u < 8 - kPolyPer8; ++u) p[u] = ex2(y[u]);
      if (kPolyPer8 >= 2) ex2_poly2(y[6], y[7], p[6], p[7]);
      if (kPolyPer8 >= 4) ex2_poly2(y[4], y[5], p[4], p[5]);
      if (MASKED) {
#pragma unroll
        for (int u = 0; u < 8; ++u) p[u] = ((word >> (q + u)) & 1u) ? p[u] : 0.f;
      }
      add2(s0, s1, s0, s1, p[0], p[1]);
      add2(s2, s3, s2, s3, p[2], p[3]);
      add2(s0, s1, s0, s1, p[4], p[5]);
      add2(s2, s3, s2, s3, p[6], p[7]);
#pragma unroll
      for (int u = 0; u < 8; u += 2) {
        __nv_bfloat162 h = __floats2bfloat162_rn(p[u], p[u + 1]);
        pk[(q + u) >> 1] = *reinterpret_cast<uint32_t*>(&h);
      }
    }
  } else {
#pragma unroll
    for (int q = 0; q < 16; ++q) pk[q] = 0u;
  }
}

template <bool MASKED>
__device__ __forceinline__ float sweep_exp(uint32_t tS, const uint4& bits, float scale, float neg_m) {
  uint32_t ra[32], rb[32];
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
  tmem_ld32(tS, ra);
  tc_wait_ld();
  // two chunks per trip (one in each register set), the loop itself is not unrolled: half the code
#pragma unroll 1
  for (int cc = 0; cc < 2; ++cc) {
    uint32_t pk[16];
    tmem_ld32(tS + (2 * cc + 1) * 32, rb);
    exp_chunk<MASKED>(ra, cc ? bits.z : bits.x, scale, neg_m, pk, s0, s1, s2, s3);
    tc_wait_ld();
    tmem_st16(tS + (2 * cc) * 16, pk);
    if (cc == 0) tmem_ld32(tS + 2 * 32, ra);
    exp_chunk<MASKED>(rb, cc ? bits.w : bits.y, scale, neg_m, pk, s0, s1, s2, s3);
    if (cc == 0) tc_wait_ld();
    tmem_st16(tS + (2 * cc + 1) * 16, pk);
  }
  return (s0 + s1) + (s2 + s3);
}

// RANGED: only the work items whose first row lies in the row range of their sequence are processed.
// D: head_dim, 128 or 64.  With 64 a Q / K / V tile is one 16 KB box of the tensor maps (the slots keep their size),
// S = Q K^T takes four MMAs instead of eight and O has 64 columns.
template <bool RANGED, int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                  const __grid_constant__ CUtensorMap tmG, const AttnParams prm) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sQ = sbase + SmemLayout::q;
  const uint32_t sSlots = sbase + SmemLayout::slots;
  const uint32_t bar0 = sbase + SmemLayout::bars;
  const uint32_t bQFull = bar0, bQEmpty = bar0 + 8;
  const uint32_t bSlotFull = bar0 + 16, bSlotEmpty = bSlotFull + 8 * kSlots;
  const uint32_t bSFull = bSlotEmpty + 8 * kSlots, bPFull = bSFull + 16, bOFinal = bPFull + 16;
  const uint32_t bSchedFull = bOFinal + 16, bSchedEmpty = bSchedFull + 16;
  volatile int* sched_items = reinterpret_cast<volatile int*>(smem + SmemLayout::sched_items);
  volatile uint32_t* step_desc = reinterpret_cast<volatile uint32_t*>(smem + SmemLayout::step_desc);
  ItemRec* item_rec = reinterpret_cast<ItemRec*>(smem + SmemLayout::item_rec);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SmemLayout::tmem_slot);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + SmemLayout::abort_flag);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned char* blob = prm.blob;
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int nitems = H->prows;
  const uint32_t* tiles = reinterpret_cast<const uint32_t*>(blob + H->off_tiles);
  // a blob with gathered-column tiles needs the larger scratch: nothing is computed without it, and the status
  // word says why (the gather kernel is not even launched when the scratch holds no tile at all)
  if ((H->flags & DAM_FLAG_GATHER) && H->attn_scratch_bytes > prm.scratch_bytes) {
    if (blockIdx.x == 0 && tid == 0) atomicMax(prm.status, (uint32_t)DAM_ERR_BUFFER_TOO_SMALL);
    return;
  }
  // Dynamic scheduling: the work list is sorted longest first; the producer thread takes positions from a
  // global counter (the first one is the CTA index) and hands each to the other roles through a two-entry
  // ring in shared memory.  A negative position ends the loop.
  auto item_active = [&](const Item& it) -> bool {
    if (!RANGED) return true;
    const int r0 = it.qb0 * DAM_TILE;
    return r0 >= __ldg(prm.ranges + 2 * it.seq) && r0 < __ldg(prm.ranges + 2 * it.seq + 1);
  };
  auto next_item_consumer = [&](uint32_t n, bool arrive) -> int {
    const uint32_t slot = n & 1u;
    if (!mbar_wait(bSchedFull + 8 * slot, (n >> 1) & 1u, abort_flag)) return -2;
    const int w = sched_items[slot];
    if (arrive) mbar_arrive(bSchedEmpty + 8 * slot);
    return w;
  };

  if (tid == 0) {
    mbar_init(bQFull, 1); mbar_init(bQEmpty, 1);
    for (int s = 0; s < kSlots; ++s) { mbar_init(bSlotFull + 8 * s, 1); mbar_init(bSlotEmpty + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bSFull + 8 * s, 1); mbar_init(bPFull + 8 * s, 4); mbar_init(bOFinal + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bSchedFull + 8 * s, 1); mbar_init(bSchedEmpty + 8 * s, 9); }   // MMA thread + 8 softmax warps
    *abort_flag = 0u;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO); tma_prefetch_desc(&tmG);
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // launched as a programmatic dependent of the kernel that gathers the matched columns: everything above ran
  // under that kernel's tail; its tiles (and the cleared work counter) are visible from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // Registers are handed out per warpgroup: the first one (one producer thread, one issuing thread) keeps 72 per
  // thread and the two softmax warpgroups take 216 each (72 * 128 + 216 * 256 = the 168 * 384 the CTA starts with).
  // With 56 the issuing thread spills and the kernel is 6 % slower; with 88 or 104 the softmax warps lose more
  // than the first warpgroup gains.
  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t sc = 0, ic = 0, step = 0;
      uint32_t armed[kSlots];
#pragma unroll
      for (int s = 0; s < kSlots; ++s) armed[s] = 2u;      // 2 = never armed
      bool ok = true;
      auto load_tile = [&](const CUtensorMap* tm, int head, int tok) -> bool {
        const uint32_t s = sc % kSlots, ph = (sc / kSlots) & 1u;
        if (!mbar_wait(bSlotEmpty + 8 * s, ph ^ 1u, abort_flag)) return false;
        const uint32_t dst = sSlots + s * kSlotBytes, bar = bSlotFull + 8 * s;
        mbar_arrive_expect_tx(bar, DAM_TILE * D * 2);
        tma_load_3d(dst, tm, bar, 0, head, tok);
        if (D == 128) tma_load_3d(dst + 16384, tm, bar, 64, head, tok);
        armed[s] = ph;
        ++sc;
        return true;
      };
      for (uint32_t n = 0; ok; ++n) {
        // claim the next position of the work list and publish it to the other roles
        const uint32_t slot = n & 1u;
        if (!(ok = mbar_wait(bSchedEmpty + 8 * slot, ((n >> 1) & 1u) ^ 1u, abort_flag))) break;
        int w = n == 0 ? (int)blockIdx.x : (int)(gridDim.x + atomicAdd(prm.work_counter, 1u));
        if (w >= nitems) w = -1;
        Item it;
        bool skip = false;
        long long gtile0 = 0;
        if (w >= 0) {
          const uint4* src = reinterpret_cast<const uint4*>(blob + H->off_work) + 2 * (size_t)w;
          const uint4 u = __ldg(src), v = __ldg(src + 1);
          it = item_from_words(u, v);
          skip = it.a0 == it.b1 || !item_active(it);         // no tile in either list, or outside the row range
          ItemRec& rec = item_rec[slot];
          rec.u = u; rec.v = v;
          if (!skip) {
            const DamSeq sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[it.seq];
            rec.eA = it.a0 < it.a1 ? __ldg(tiles + it.a0) : 0u;
            rec.eB = it.b0 < it.b1 ? __ldg(tiles + it.b0) : 0u;
            rec.hb = dam_head_bits(blob, H, sq, it.head);
            // gathered-column tiles of this (sequence, head): K tile at rows (2T) * 128, V tile at (2T + 1) * 128
            gtile0 = (long long)sq.gath_off + (long long)it.head * sq.nL;
          }
        }
        // the entry tells the MMA thread whether the item has steps at all, so that it never reads the work list
        sched_items[slot] = w < 0 ? w : (w | (skip ? kSchedNoSteps : 0));
        mbar_arrive(bSchedFull + 8 * slot);
        if (w < 0) break;
        if (skip) continue;
        if (!(ok = mbar_wait(bQEmpty, (ic & 1u) ^ 1u, abort_flag))) break;
        const int tokq = it.tok0 + it.qb0 * DAM_TILE;
        mbar_arrive_expect_tx(bQFull, (it.hasB ? 2 : 1) * DAM_TILE * D * 2);
        tma_load_3d(sQ, &tmQ, bQFull, 0, it.head, tokq);
        if (D == 128) tma_load_3d(sQ + 16384, &tmQ, bQFull, 64, it.head, tokq);
        if (it.hasB) {
          tma_load_3d(sQ + 32768, &tmQ, bQFull, 0, it.head, tokq + DAM_TILE);
          if (D == 128) tma_load_3d(sQ + 49152, &tmQ, bQFull, 64, it.head, tokq + DAM_TILE);
        }
        ++ic;
        const int kvh = it.head / prm.group;
        Walker wk; wk.init(tiles, it);
        int kb; uint32_t kA, kB;
        while (ok && wk.next(kb, kA, kB)) {
          // what the MMA thread needs to know about this step, visible to it once the step's K tile has landed
          step_desc[step++ & 15u] = (kA ? kStepA : 0u) | (kB ? kStepB : 0u) | (kA && wk.a_done() ? kStepLastA : 0u) |
                                    (kB && wk.b_done() ? kStepLastB : 0u) | (wk.a_done() && wk.b_done() ? 0u : kStepMore);
          if (kA == DAM_KIND_GATHERED || kB == DAM_KIND_GATHERED) {
            const int row = (int)((gtile0 + kb) * 2 * DAM_TILE);
            ok = load_tile(&tmG, 0, row);
            if (ok) ok = load_tile(&tmG, 0, row + DAM_TILE);
          } else {
            ok = load_tile(&tmK, kvh, it.tok0 + kb * DAM_TILE);
            if (ok) ok = load_tile(&tmV, kvh, it.tok0 + kb * DAM_TILE);
          }
        }
      }
      if (!ok) {
        // drain: copies already issued still write into shared memory; wait for them (bounded)
        uint32_t dummy = 0;
        for (int s = 0; s < kSlots; ++s)
          if (armed[s] != 2u) mbar_wait(bSlotFull + 8 * s, armed[s], &dummy, 20000000ull);
        mbar_wait(bQFull, (ic + 1u) & 1u, &dummy, 20000000ull);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_qk = idesc_bf16_f32(128, 128, 0);
      const uint32_t idesc_pv = idesc_bf16_f32(128, D, 1);
      uint32_t sc = 0, ic = 0, step = 0;
      uint32_t cP[2] = {0u, 0u};           // P tiles consumed per stream (phase of p_full)
      bool ok = true;
      // descriptors: the high words are invariant, the low words step by (byte offset >> 4)
      const uint64_t dQ = smem_desc_sw128(sQ, 16, 1024);
      const uint64_t dK = smem_desc_sw128(sSlots, 16, 1024);
      const uint64_t dV = smem_desc_sw128(sSlots, 16384, 1024);
      const uint32_t dQ_lo = (uint32_t)dQ, dQ_hi = (uint32_t)(dQ >> 32);
      const uint32_t dK_lo = (uint32_t)dK, dK_hi = (uint32_t)(dK >> 32);
      const uint32_t dV_lo = (uint32_t)dV, dV_hi = (uint32_t)(dV >> 32);
      auto issue_s = [&](int X, uint32_t slot) {
        const uint32_t a0 = dQ_lo + X * (kSlotBytes >> 4), b0 = dK_lo + slot * (kSlotBytes >> 4);
        const uint32_t d = tmem + kColS + X * 128;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
          mma_ss_lh(d, a0 + off, dQ_hi, b0 + off, dK_hi, idesc_qk, ks > 0 ? 1u : 0u);
        }
        tc_commit(bSFull + 8 * X);
      };
      auto issue_pv = [&](int X, uint32_t slot, bool accumulate) -> bool {
        if (!mbar_wait(bPFull + 8 * X, cP[X] & 1u, abort_flag)) return false;
        ++cP[X];
        tc_fence_after();
        const uint32_t b0 = dV_lo + slot * (kSlotBytes >> 4);
        const uint32_t d = tmem + kColO + X * 128, a = tmem + kColS + X * 128;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          // V is MN-major: 16 keys per step = 2048 bytes; 64-column halves 16384 bytes apart
          mma_ts_lh(d, a + ks * 8, b0 + ks * (2048 >> 4), dV_hi, idesc_pv, (accumulate || ks > 0) ? 1u : 0u);
        }
        return true;
      };
      for (uint32_t n = 0; ok; ++n) {
        const int w = next_item_consumer(n, true);
        if (w < 0) { ok = (w == -1); break; }
        if (w & kSchedNoSteps) continue;
        if (!(ok = mbar_wait(bQFull, ic & 1u, abort_flag))) break;
        ++ic;
        // S of the first step (the producer's descriptor of a step is readable once its K tile is)
        uint32_t d;
        {
          const uint32_t s = sc % kSlots;
          if (!(ok = mbar_wait(bSlotFull + 8 * s, (sc / kSlots) & 1u, abort_flag))) break;
          d = step_desc[step & 15u];
          tc_fence_after();
          if (d & kStepA) issue_s(0, s);
          if (d & kStepB) issue_s(1, s);
          tc_commit(bSlotEmpty + 8 * s);
          ++sc;
        }
        bool accA = false, accB = false;
        while (ok) {
          const bool have_nxt = (d & kStepMore) != 0u;
          if (!have_nxt) tc_commit(bQEmpty);                   // every S of this item has been issued
          const uint32_t sv = sc % kSlots;                     // V of the current step
          if (!(ok = mbar_wait(bSlotFull + 8 * sv, (sc / kSlots) & 1u, abort_flag))) break;
          ++sc;
          uint32_t sk = 0, dn = 0;
          // a stream's output is final right after the P V of its last listed tile
          if (d & kStepA) { if (!(ok = issue_pv(0, sv, accA))) break; accA = true; if (d & kStepLastA) tc_commit(bOFinal); }
          if (have_nxt) {                                      // K of the next step
            sk = sc % kSlots;
            if (!(ok = mbar_wait(bSlotFull + 8 * sk, (sc / kSlots) & 1u, abort_flag))) break;
            ++sc;
            dn = step_desc[(step + 1u) & 15u];
            tc_fence_after();
            if (dn & kStepA) issue_s(0, sk);
          }
          if (d & kStepB) { if (!(ok = issue_pv(1, sv, accB))) break; accB = true; if (d & kStepLastB) tc_commit(bOFinal + 8); }
          tc_commit(bSlotEmpty + 8 * sv);
          ++step;
          if (!have_nxt) break;
          if (dn & kStepB) issue_s(1, sk);
          tc_commit(bSlotEmpty + 8 * sk);
          d = dn;
        }
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    // ------------------------------------------------------------------ softmax / epilogue warps
    const int X = (warp - 4) >> 2;                           // stream: 0 = block 2p, 1 = block 2p+1
    const int r = (warp & 3) * 32 + lane;                    // row of the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_addr + kColS + X * 128;
    const uint32_t tO = tmem + lane_addr + kColO + X * 128;
    const uint32_t bS = bSFull + 8 * X, bP = bPFull + 8 * X, bO = bOFinal + 8 * X;
    const uint32_t stage_addr = sbase + SmemLayout::stage + X * kStageBytes + (warp & 3) * 4096;   // 32 rows x 128 B
    uint32_t cS = 0, cO = 0;
    bool ok = true;
    for (uint32_t n = 0; ok; ++n) {
      const int ws = next_item_consumer(n, false);
      if (ws < 0) {
        __syncwarp();
        if (lane == 0 && ws != -2) mbar_arrive(bSchedEmpty + 8 * (n & 1u));
        ok = (ws == -1);
        break;
      }
      const ItemRec& rec = item_rec[n & 1u];
      const Item it = item_from_words(rec.u, rec.v);
      const DamHeadBits hb = rec.hb;                         // (not meaningful for an item without steps)
      const uint32_t e_first = X ? rec.eB : rec.eA;
      __syncwarp();
      if (lane == 0) mbar_arrive(bSchedEmpty + 8 * (n & 1u));               // the whole warp has read the record
      if ((X == 1 && !it.hasB) || !item_active(it)) continue;
      const int qb = it.qb0 + X;
      const uint32_t t0 = X ? it.b0 : it.a0, t1 = X ? it.b1 : it.a1;
      const int i = qb * DAM_TILE + r;
      const bool row_valid = i < it.S;
      __nv_bfloat16* orow = prm.O + (int64_t)(it.tok0 + i) * prm.o_stride_tok + (int64_t)it.head * prm.o_stride_head;
      float* lse_p = prm.lse + (int64_t)it.head * prm.total_tokens + it.tok0 + i;
      if (t0 == t1) {
        if (row_valid) {
          const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
          for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = z;
          *lse_p = -CUDART_INF_F;
        }
        continue;
      }
      float m_ref = -CUDART_INF_F;   // reference max (scaled, log2 domain) that P and O are expressed against
      float l = 0.f;
      // the mask words of a tile come from global memory: they are fetched one tile ahead
      auto tile_bits = [&](uint32_t e, bool& need) -> uint4 {
        const uint32_t kind = e >> 28;
        if (kind == DAM_KIND_GATHERED) {       // all rows see the same columns: the first n of the tile
          const int n = (int)((e >> 16) & 0xFFu) + 1;
          need = n < DAM_TILE;
          return row_valid ? dam_low_ones128(n) : make_uint4(0u, 0u, 0u, 0u);
        }
        const int kb = (int)(e & 0x0FFFFFFFu);
        need = (kind != DAM_KIND_FULL) || (prm.causal && kb >= qb) || ((kb + 1) * DAM_TILE > it.S);
        return need ? dam_apply_bits(hb, kind, i, kb, prm.causal) : make_uint4(~0u, ~0u, ~0u, ~0u);
      };
      uint32_t e_next = t0 + 1 < t1 ? __ldg(tiles + t0 + 1) : 0u;
      bool need_nx = false;
      uint4 bits_nx = tile_bits(e_first, need_nx);
      for (uint32_t t = t0; t < t1; ++t) {
        const bool need_mask = need_nx;
        const uint4 bits = bits_nx;
        if (t + 1 < t1) {
          bits_nx = tile_bits(e_next, need_nx);
          if (t + 2 < t1) e_next = __ldg(tiles + t + 2);
        }
        if (!(ok = mbar_wait(bS, cS & 1u, abort_flag))) break;
        ++cS;
        tc_fence_after();
        // ---- sweep 1: row maximum of the raw dot products.  On a masked tile the maximum over all entries is
        //      tried first: it bounds the masked one from above, so when it does not exceed the reference by more
        //      than the threshold for any row of the warp, the reference stays where it is and the masked
        //      maximum (two more instructions per element) is never needed.  The result is the same either way.
        bool masked_max = need_mask && (t == t0);            // the first tile sets the reference
        float mx = -CUDART_INF_F;
        if (!masked_max) {
          const float mu = sweep_max<false>(tS, bits);
          if (!need_mask) mx = mu;
          else masked_max = __any_sync(0xFFFFFFFFu, mu * prm.scale_log2 - m_ref > kRescaleThreshold);   // -inf reference: true
        }
        if (masked_max) mx = sweep_max<true>(tS, bits);
        const float m_new = fmaxf(m_ref, mx * prm.scale_log2);
        // move the reference only on the first tile or when the max grew by more than the threshold
        bool move = (t == t0) || (m_new - m_ref > kRescaleThreshold);   // -inf reference: inf > 8 is true
        if (m_new == -CUDART_INF_F) move = false;
        float alpha = 1.f;
        if (move) {
          alpha = (m_ref == -CUDART_INF_F) ? 0.f : ex2(m_ref - m_new);
          m_ref = m_new;
        }
        const float mm = (m_ref == -CUDART_INF_F) ? 0.f : m_ref;
        // ---- sweep 2: probabilities against the reference max, packed to bf16 into the first half of S
        const float tsum = need_mask ? sweep_exp<true>(tS, bits, prm.scale_log2, -mm)
                                     : sweep_exp<false>(tS, bits, prm.scale_log2, -mm);
        l = l * alpha + tsum;
        // ---- O is complete up to the previous tile of this stream (its MMAs precede S of this tile)
        if (t > t0) {
          const bool resc = alpha != 1.f;
          if (__any_sync(0xFFFFFFFFu, resc)) {
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t rr[32];
              tmem_ld32(tO + c * 32, rr);
              tc_wait_ld();
#pragma unroll
              for (int q = 0; q < 32; ++q) rr[q] = __float_as_uint(__uint_as_float(rr[q]) * alpha);
              tmem_st32(tO + c * 32, rr);
            }
          }
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bP);
      }
      if (!ok) break;
      // ---- epilogue: O / l and the log-sum-exp
      if (!(ok = mbar_wait(bO, cO & 1u, abort_flag))) break;
      ++cO;
      tc_fence_after();
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      if ((qb + 1) * DAM_TILE <= it.S) {
        // whole tile inside the sequence: through shared memory (128-byte swizzle) and TMA stores
        const int tok = it.tok0 + qb * DAM_TILE;
#pragma unroll
        for (int half = 0; half < D / 64; ++half) {
          uint32_t pk[32];
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t rr[32];
            tmem_ld32(tO + (half * 2 + c) * 32, rr);
            tc_wait_ld();
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              __nv_bfloat162 hpair = __floats2bfloat162_rn(__uint_as_float(rr[2 * q]) * inv, __uint_as_float(rr[2 * q + 1]) * inv);
              pk[c * 16 + q] = *reinterpret_cast<uint32_t*>(&hpair);
            }
          }
          // every warp stages and stores its own 32 rows: no synchronisation beyond the warp.  The warp's
          // staging block is free once its previous store has been read out of shared memory.
          if (lane == 0) tma_store_wait_read();
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t dst = stage_addr + lane * 128 + ((j ^ (lane & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pk[4 * j]), "r"(pk[4 * j + 1]),
                         "r"(pk[4 * j + 2]), "r"(pk[4 * j + 3]) : "memory");
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(&tmO, stage_addr, half * 64, it.head, tok + (warp & 3) * 32);
            tma_store_commit();
          }
        }
      } else {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t rr[32];
          tmem_ld32(tO + c * 32, rr);
          tc_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
              uint32_t o[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                __nv_bfloat162 hpair = __floats2bfloat162_rn(__uint_as_float(rr[v4 * 8 + 2 * q]) * inv,
                                                             __uint_as_float(rr[v4 * 8 + 2 * q + 1]) * inv);
                o[q] = *reinterpret_cast<uint32_t*>(&hpair);
              }
              reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
        }
      }
      if (row_valid) *lse_p = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -CUDART_INF_F;
      tc_fence_before();
    }
    if (lane == 0) tma_store_wait_all();                    // outstanding O stores complete before the CTA exits
  }

  if (*abort_flag && tid == 64) atomicMax(prm.status, (uint32_t)DAM_ERR_DEVICE_TIMEOUT);
  if (blockIdx.x == 0 && tid == 64) prm.status[3] = 1u;      // word 4 of the scratch block: which kernel served the call
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// Copies the K and V rows of the matched columns of every (sequence, head) into dense tiles of 128 keys in
// the scratch buffer (K tile at rows (2T) * 128, V tile at rows (2T + 1) * 128 of a [rows][head_dim] bf16 array;
// T = gath_off + head * nL + g).  Rows past the last matched column are zero.  One block per tile, grid-stride.
__global__ void __launch_bounds__(128)
gather_columns_kernel(const unsigned char* __restrict__ blob, const __nv_bfloat16* __restrict__ K,
                      const __nv_bfloat16* __restrict__ V, int Hq, int group, int d, int64_t kst, int64_t ksh, int64_t vst,
                      int64_t vsh, unsigned char* scratch, unsigned long long scratch_bytes) {
  asm volatile("griddepcontrol.launch_dependents;");     // the attention kernel behind this one may start its prologue
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  if (!(H->flags & DAM_FLAG_GATHER)) return;
  if (H->attn_scratch_bytes > scratch_bytes) {
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicMax(reinterpret_cast<uint32_t*>(scratch) + 1, (uint32_t)DAM_ERR_BUFFER_TOO_SMALL);
    return;
  }
  __shared__ int pref[1025];
  __shared__ int col[DAM_TILE];
  uint4* out = reinterpret_cast<uint4*>(scratch + 256);
  const DamSeq* seqs = reinterpret_cast<const DamSeq*>(blob + H->off_seq);
  const int tid = threadIdx.x;
  for (long long T = blockIdx.x; T < (long long)H->gath_tiles; T += gridDim.x) {
    int b = 0;
    while (b + 1 < H->num_seqs && (long long)seqs[b + 1].gath_off <= T) ++b;
    const DamSeq sq = seqs[b];
    if (sq.nL == 0) continue;
    const int h = (int)((T - (long long)sq.gath_off) / sq.nL), g = (int)((T - (long long)sq.gath_off) % sq.nL);
    if (h >= Hq) continue;
    const uint32_t* Vw = reinterpret_cast<const uint32_t*>(blob + H->off_dv) + sq.dv_off + (uint64_t)h * 3 * sq.W + 2 * sq.W;
    // exclusive prefix popcounts of the V words (W <= 1024 words, i.e. windows up to 32768 tokens)
    const int W = min(sq.W, 1024);
    __syncthreads();
    if (tid < 32) {                                              // warp 0: 32 words per step
      int run = 0;
      for (int w0 = 0; w0 < W; w0 += 32) {
        const int w = w0 + tid;
        const int pc = w < W ? __popc(__ldg(Vw + w)) : 0;
        int inc = pc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
          if (tid >= o) inc += y;
        }
        if (w < W) pref[w] = run + inc - pc;
        run += __shfl_sync(0xFFFFFFFFu, inc, 31);
      }
      if (tid == 0) pref[W] = run;
    }
    __syncthreads();
    const int nV = pref[W];
    if (g * DAM_TILE >= nV) continue;                         // capacity tile that no row list refers to
    {
      const int rank = g * DAM_TILE + tid;
      int c = -1;
      if (rank < nV) {
        int lo = 0, hi = W;                                     // last word with pref <= rank
        while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (pref[mid] <= rank) lo = mid; else hi = mid; }
        c = lo * 32 + (int)__fns(Vw[lo], 0, rank - pref[lo] + 1);
      }
      col[tid] = c;
    }
    __syncthreads();
    const __nv_bfloat16* Kh = K + (int64_t)sq.tok_start * kst + (int64_t)(h / group) * ksh;
    const __nv_bfloat16* Vh = V + (int64_t)sq.tok_start * vst + (int64_t)(h / group) * vsh;
    const int ppr = d >> 3;                                      // 16-byte pieces per row (16 at head_dim 128, 8 at 64)
    const int part = tid % ppr, r0 = tid / ppr, step = 128 / ppr;
    // eight rows of K and of V per thread are requested before the first is stored (the block is one dependent
    // chain of loads as it is; one round trip per row would be most of its time)
    for (int rb = r0; rb < DAM_TILE; rb += 8 * step) {
      uint4 kv[8], vv[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int r = rb + u * step;
        const int c = r < DAM_TILE ? col[r] : -1;
        kv[u] = make_uint4(0u, 0u, 0u, 0u); vv[u] = kv[u];
        if (c >= 0) {
          kv[u] = __ldg(reinterpret_cast<const uint4*>(Kh + (int64_t)c * kst) + part);
          vv[u] = __ldg(reinterpret_cast<const uint4*>(Vh + (int64_t)c * vst) + part);
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int r = rb + u * step;
        if (r < DAM_TILE) {
          out[((size_t)(2 * T) * DAM_TILE + r) * ppr + part] = kv[u];
          out[((size_t)(2 * T + 1) * DAM_TILE + r) * ppr + part] = vv[u];
        }
      }
    }
  }
}

// Self-test of the bounded wait every kernel in this library uses: waits on an mbarrier that nothing ever
// arrives on, with the given limit; the wait gives up, the status word is set and the kernel returns normally.
__global__ void bounded_wait_selftest_kernel(uint32_t* status, unsigned long long limit_ns, unsigned long long* waited_ns) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0u;
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint64_t t0 = globaltimer_ns();
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, limit_ns);
    *waited_ns = globaltimer_ns() - t0;
    if (!ok) atomicMax(status, (uint32_t)DAM_ERR_DEVICE_TIMEOUT);
  }
}

}  // namespace

cudaError_t dam_launch_bounded_wait_selftest(void* scratch, unsigned long long limit_ns, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(reinterpret_cast<uint32_t*>(scratch) + 1, limit_ns,
                                                  reinterpret_cast<unsigned long long*>(scratch) + 1);
  return cudaGetLastError();
}

cudaError_t dam_launch_attn_sm100(const void* Q, const void* K, const void* V, const void* blob,
                                  const dam_shape_t* s, int causal, float scale, void* O, float* lse, void* scratch,
                                  size_t scratch_bytes, const int32_t* ranges, bool run_gather, cudaStream_t st) {
  const int d = s->head_dim;
  if (s->dtype != DAM_BF16 || (d != 128 && d != 64)) return cudaErrorNotSupported;
  if (s->total_tokens == 0) return cudaSuccess;
  int dev = 0;
  DamDeviceInfo di;
  cudaError_t e;
  if ((e = dam_current_device(&dev, &di)) != cudaSuccess) return e;
  if (di.cc_major != 10 || di.smem_optin < kSmemBytes) return cudaErrorNotSupported;
  if ((e = dam_device_table().once(dev, DAM_SETUP_ATTN_SMEM, [](void) -> cudaError_t {
         cudaError_t r;
         if ((r = cudaFuncSetAttribute(attn_sm100_kernel<false, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return r;
         if ((r = cudaFuncSetAttribute(attn_sm100_kernel<true, 128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return r;
         if ((r = cudaFuncSetAttribute(attn_sm100_kernel<false, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess) return r;
         return cudaFuncSetAttribute(attn_sm100_kernel<true, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
       })) != cudaSuccess)
    return e;
  const int sm_count = di.sm_count;
  // gathered-column tiles (if the blob has any) live after the 256-byte status block of the scratch buffer
  const size_t grows = scratch_bytes > 256 ? (scratch_bytes - 256) / (size_t)(d * 2) : 0;      // rows of head_dim bf16
  CUtensorMap tq, tk, tv, to, tg;
  const bool has_g = grows >= 2 * DAM_TILE;
  if (!dam_make_tmap_bf16(&tg, has_g ? reinterpret_cast<const unsigned char*>(scratch) + 256 : Q, d, 1,
                          has_g ? (int64_t)grows : DAM_TILE, d, d))
    return cudaErrorInvalidValue;
  if (has_g && run_gather) {
    gather_columns_kernel<<<sm_count * 4, 128, 0, st>>>(
        reinterpret_cast<const unsigned char*>(blob), reinterpret_cast<const __nv_bfloat16*>(K),
        reinterpret_cast<const __nv_bfloat16*>(V), s->num_q_heads, s->num_q_heads / s->num_kv_heads, d, s->k_stride_tok,
        s->k_stride_head, s->v_stride_tok, s->v_stride_head, reinterpret_cast<unsigned char*>(scratch),
        (unsigned long long)scratch_bytes);
  }
  if (!dam_make_tmap_bf16(&to, O, d, s->num_q_heads, s->total_tokens, s->o_stride_tok, s->o_stride_head, 32) ||
      !dam_make_tmap_bf16(&tq, Q, d, s->num_q_heads, s->total_tokens, s->q_stride_tok, s->q_stride_head) ||
      !dam_make_tmap_bf16(&tk, K, d, s->num_kv_heads, s->total_tokens, s->k_stride_tok, s->k_stride_head) ||
      !dam_make_tmap_bf16(&tv, V, d, s->num_kv_heads, s->total_tokens, s->v_stride_tok, s->v_stride_head))
    return cudaErrorInvalidValue;
  int pairs = 0;
  for (int b = 0; b < s->num_seqs; ++b) {
    int nq = (s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b] + DAM_TILE - 1) / DAM_TILE;
    pairs += (nq + 1) / 2;
  }
  pairs *= s->num_q_heads;
  if (pairs == 0) return cudaSuccess;
  AttnParams p;
  p.blob = reinterpret_cast<const unsigned char*>(blob);
  p.O = reinterpret_cast<__nv_bfloat16*>(O);
  p.lse = lse;
  p.status = reinterpret_cast<uint32_t*>(scratch) + 1;
  p.work_counter = reinterpret_cast<uint32_t*>(scratch) + 2;
  p.scratch_bytes = scratch_bytes;
  p.ranges = ranges;
  p.Hq = s->num_q_heads; p.group = s->num_q_heads / s->num_kv_heads; p.total_tokens = s->total_tokens;
  p.causal = causal;
  p.o_stride_tok = s->o_stride_tok; p.o_stride_head = s->o_stride_head;
  p.scale_log2 = scale * 1.4426950408889634f;
  const int grid = pairs < sm_count ? pairs : sm_count;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (d == 128) {
    if (ranges) return cudaLaunchKernelEx(&cfg, attn_sm100_kernel<true, 128>, tq, tk, tv, to, tg, p);
    return cudaLaunchKernelEx(&cfg, attn_sm100_kernel<false, 128>, tq, tk, tv, to, tg, p);
  }
  if (ranges) return cudaLaunchKernelEx(&cfg, attn_sm100_kernel<true, 64>, tq, tk, tv, to, tg, p);
  return cudaLaunchKernelEx(&cfg, attn_sm100_kernel<false, 64>, tq, tk, tv, to, tg, p);
}
