// Window scoring on the 5th-generation tensor cores (sm_100a): bf16 inputs, head_dim 128 or 64 (template parameter:
// with 64 a Q / K tile is one 16 KB box of the tensor maps and S = Q K^T takes four MMAs instead of eight).
//
// For every (sequence, query head) the causal softmax map over the first L tokens is computed tile by
// tile and thresholded straight into the bit-packed true mask (paper Sec. 4.2.1 - 4.2.3); the map itself
// is never stored unless the caller asks for the fp32 dump.  Four S buffers in TMEM let the MMA warp run two
// tiles ahead of each softmax group.  A work item is one 128-row query block of
// one (sequence, head).  Two sweeps over its kv tiles kb = 0 .. qb:
//   sweep A  S = Q K^T (tcgen05, accumulator in TMEM) -> per-row running max and sum;
//   sweep B  S again -> p = exp2(x - max) / sum in fp32 -> bit = [p >= p*] -> one 16-byte store of the
//            row's 128 bits per tile (and the optional dump of p).
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-17 four groups of one thread per query row;
// group G owns TMEM buffer G, i.e. every fourth kv tile, and the groups merge their row statistics through
// shared memory between the sweeps.  Every wait is bounded.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "dam_internal.cuh"
#include "sm100_ptx.cuh"

using namespace sm100;

namespace {

constexpr int kSlots = 5;
constexpr int kSlotBytes = 32768;
constexpr int kThreads = 576;              // producer warp, MMA warp, four softmax groups of four warps
constexpr uint32_t kTmemCols = 512;       // four S buffers: tile g uses buffer g & 3, which softmax group g & 3 owns

struct SmemLayout {
  static constexpr int q = 0;
  static constexpr int slots = kSlotBytes;
  static constexpr int bars = kSlotBytes * (1 + kSlots);
  // q_full, q_empty, slot_full[kSlots], slot_empty[kSlots], s_full[4], s_empty[4], stat_ready,
  // sched_full[2], sched_empty[2]
  static constexpr int n_bars = 2 + 2 * kSlots + 13;
  static constexpr int sched_items = bars + 8 * n_bars;     // int[2]
  static constexpr int stat = sched_items + 8;              // float2 [2][4][128]
  static constexpr int tmem_slot = stat + 2 * 4 * 128 * 8;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int total = abort_flag + 4;
};
constexpr int kSmemBytes = SmemLayout::total + 1024;

struct ScoreParams {
  unsigned char* blob;
  float* dump;
  uint32_t* status;
  uint32_t* work_counter;     // zero at launch
  int num_seqs, Hq, group, max_nL;
  float scale_log2, pstar;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

struct Item { int b, h, qb, valid; DamSeq sq; };

__device__ __forceinline__ Item decode_item(const unsigned char* blob, const DamHeader* H, const ScoreParams& p, int w) {
  Item it;
  const int per = p.num_seqs * p.Hq;
  it.qb = p.max_nL - 1 - w / per;           // heaviest query blocks first
  const int sh = w % per;
  it.b = sh / p.Hq; it.h = sh % p.Hq;
  it.sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[it.b];
  it.valid = it.qb < it.sq.nL;
  return it;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
score_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const ScoreParams prm) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sQ = sbase + SmemLayout::q;
  const uint32_t sSlots = sbase + SmemLayout::slots;
  const uint32_t bar0 = sbase + SmemLayout::bars;
  const uint32_t bQFull = bar0, bQEmpty = bar0 + 8;
  const uint32_t bSlotFull = bar0 + 16, bSlotEmpty = bSlotFull + 8 * kSlots;
  const uint32_t bSFull = bSlotEmpty + 8 * kSlots, bSEmpty = bSFull + 32, bStat = bSEmpty + 32;
  const uint32_t bSchedFull = bStat + 8, bSchedEmpty = bSchedFull + 16;
  volatile int* sched_items = reinterpret_cast<volatile int*>(smem + SmemLayout::sched_items);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SmemLayout::tmem_slot);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + SmemLayout::abort_flag);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* blob = prm.blob;
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int nitems = prm.max_nL * prm.num_seqs * prm.Hq;
  // Items (heaviest query blocks first) are claimed from a global counter by the producer thread and handed
  // to the MMA thread and the eight softmax warps through a two-entry ring; a negative entry ends the loop.
  auto next_item_consumer = [&](uint32_t n) -> int {
    const uint32_t slot = n & 1u;
    if (!mbar_wait(bSchedFull + 8 * slot, (n >> 1) & 1u, abort_flag)) return -2;
    return sched_items[slot];
  };

  if (tid == 0) {
    mbar_init(bQFull, 1); mbar_init(bQEmpty, 1);
    for (int s = 0; s < kSlots; ++s) { mbar_init(bSlotFull + 8 * s, 1); mbar_init(bSlotEmpty + 8 * s, 1); }
    for (int s = 0; s < 4; ++s) { mbar_init(bSFull + 8 * s, 1); mbar_init(bSEmpty + 8 * s, 4); }
    mbar_init(bStat, 16);
    for (int s = 0; s < 2; ++s) { mbar_init(bSchedFull + 8 * s, 1); mbar_init(bSchedEmpty + 8 * s, 17); }   // MMA thread + 16 softmax warps
    *abort_flag = 0u;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK);
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // everything above is independent of the kernel before this one; the blob it initialises is read from here on
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (blockIdx.x == 0 && tid == 0) const_cast<DamHeader*>(H)->reserved[0] = 1ull;   // the map of this blob was scored on the tensor cores

  if (warp == 0) {
    if (lane == 0) {
      uint32_t sc = 0, ic = 0;
      uint32_t armed[kSlots];
#pragma unroll
      for (int s = 0; s < kSlots; ++s) armed[s] = 2u;
      bool ok = true;
      for (uint32_t n = 0; ok; ++n) {
        const uint32_t sl = n & 1u;
        if (!(ok = mbar_wait(bSchedEmpty + 8 * sl, ((n >> 1) & 1u) ^ 1u, abort_flag))) break;
        int w = n == 0 ? (int)blockIdx.x : (int)(gridDim.x + atomicAdd(prm.work_counter, 1u));
        if (w >= nitems) w = -1;
        sched_items[sl] = w;
        mbar_arrive(bSchedFull + 8 * sl);
        if (w < 0) break;
        const Item it = decode_item(blob, H, prm, w);
        if (!it.valid) continue;
        if (!(ok = mbar_wait(bQEmpty, (ic & 1u) ^ 1u, abort_flag))) break;
        mbar_arrive_expect_tx(bQFull, DAM_TILE * D * 2);
        const int tokq = it.sq.tok_start + it.qb * DAM_TILE;
        tma_load_3d(sQ, &tmQ, bQFull, 0, it.h, tokq);
        if (D == 128) tma_load_3d(sQ + 16384, &tmQ, bQFull, 64, it.h, tokq);
        ++ic;
        const int kvh = it.h / prm.group;
        const int ntile = 2 * (it.qb + 1);
        for (int t = 0; t < ntile && ok; ++t) {
          const int kb = t % (it.qb + 1);
          const uint32_t s = sc % kSlots, ph = (sc / kSlots) & 1u;
          if (!(ok = mbar_wait(bSlotEmpty + 8 * s, ph ^ 1u, abort_flag))) break;
          const uint32_t dst = sSlots + s * kSlotBytes, bar = bSlotFull + 8 * s;
          mbar_arrive_expect_tx(bar, DAM_TILE * D * 2);
          tma_load_3d(dst, &tmK, bar, 0, kvh, it.sq.tok_start + kb * DAM_TILE);
          if (D == 128) tma_load_3d(dst + 16384, &tmK, bar, 64, kvh, it.sq.tok_start + kb * DAM_TILE);
          armed[s] = ph;
          ++sc;
        }
      }
      if (!ok) {
        uint32_t dummy = 0;
        for (int s = 0; s < kSlots; ++s)
          if (armed[s] != 2u) mbar_wait(bSlotFull + 8 * s, armed[s], &dummy, 20000000ull);
        mbar_wait(bQFull, (ic + 1u) & 1u, &dummy, 20000000ull);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, 128, 0);
      const uint64_t dQ = smem_desc_sw128(sQ, 16, 1024), dK = smem_desc_sw128(sSlots, 16, 1024);
      const uint32_t dQ_lo = (uint32_t)dQ, dQ_hi = (uint32_t)(dQ >> 32), dK_lo = (uint32_t)dK, dK_hi = (uint32_t)(dK >> 32);
      uint32_t sc = 0, ic = 0, g = 0;
      bool ok = true;
      for (uint32_t n = 0; ok; ++n) {
        const int w = next_item_consumer(n);
        if (w != -2) mbar_arrive(bSchedEmpty + 8 * (n & 1u));
        if (w < 0) { ok = (w == -1); break; }
        const Item it = decode_item(blob, H, prm, w);
        if (!it.valid) continue;
        if (!(ok = mbar_wait(bQFull, ic & 1u, abort_flag))) break;
        ++ic;
        const int ntile = 2 * (it.qb + 1);
        for (int t = 0; t < ntile && ok; ++t, ++g, ++sc) {
          const uint32_t buf = g & 3u, s = sc % kSlots;
          if (!(ok = mbar_wait(bSEmpty + 8 * buf, ((g >> 2) & 1u) ^ 1u, abort_flag))) break;
          if (!(ok = mbar_wait(bSlotFull + 8 * s, (sc / kSlots) & 1u, abort_flag))) break;
          tc_fence_after();
          const uint32_t b0 = dK_lo + s * (kSlotBytes >> 4);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const uint32_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
            mma_ss_lh(tmem + buf * 128, dQ_lo + off, dQ_hi, b0 + off, dK_hi, idesc, ks > 0 ? 1u : 0u);
          }
          tc_commit(bSlotEmpty + 8 * s);
          tc_commit(bSFull + 8 * buf);
          if (t + 1 == ntile) tc_commit(bQEmpty);
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- row statistics and thresholding
    // Two groups of four warps; group G owns the S buffer G, i.e. every other kv tile of the item.
    const int G = (warp - 2) >> 2;
    const int r = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS0 = tmem + lane_addr;
    float2* stat = reinterpret_cast<float2*>(smem + SmemLayout::stat);      // [2 item parities][2 groups][128 rows]
    uint32_t g = 0, cG = 0, nitem = 0;      // g: tiles issued so far (all groups); cG: tiles this group consumed
    bool ok = true;
    for (uint32_t n = 0; ok; ++n) {
      const int w = next_item_consumer(n);
      __syncwarp();
      if (lane == 0 && w != -2) mbar_arrive(bSchedEmpty + 8 * (n & 1u));
      if (w < 0) { ok = (w == -1); break; }
      const Item it = decode_item(blob, H, prm, w);
      if (!it.valid) continue;
      const int L = it.sq.L, W = it.sq.W;
      const int i = it.qb * DAM_TILE + r;
      const bool row_valid = i < L;
      uint32_t* Mrow = reinterpret_cast<uint32_t*>(blob + H->off_true) + it.sq.true_off + (uint64_t)it.h * L * W + (size_t)i * W;
      float* Prow = prm.dump ? prm.dump + it.sq.p_off + (uint64_t)it.h * L * L + (size_t)i * L : nullptr;
      const int nk = it.qb + 1;
      float m = -CUDART_INF_F, l = 0.f, inv_l = 0.f, thr_raw = 0.f;
      for (int t = 0; t < 2 * nk; ++t, ++g) {
        if (t == nk) {
          // all groups have finished sweep A: merge their (max, sum) per row through shared memory
          float2* base = stat + (nitem & 1u) * 4 * DAM_TILE;
          base[G * DAM_TILE + r] = make_float2(m, l);
          __syncwarp();
          if (lane == 0) mbar_arrive(bStat);                       // release: the warp's 32 rows are written
          if (!(ok = mbar_wait(bStat, nitem & 1u, abort_flag))) break;
          float mn = m;
#pragma unroll
          for (int q = 0; q < 4; ++q) mn = fmaxf(mn, base[q * DAM_TILE + r].x);
          float ls = 0.f;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float2 o = base[q * DAM_TILE + r];
            ls += (o.x == -CUDART_INF_F) ? 0.f : o.y * ex2(o.x - mn);
          }
          m = mn; l = ls;
          inv_l = l > 0.f ? 1.0f / l : 0.f;
          thr_raw = (log2f(prm.pstar * l) - 0.03125f + m) / prm.scale_log2;   // the same bound on the raw dot product
        }
        if ((g & 3u) != (uint32_t)G) continue;
        const int kb = t % nk;
        const bool sweepB = t >= nk;
        const uint32_t buf = (uint32_t)G;
        const uint32_t tS = tS0 + buf * 128;
        if (!(ok = mbar_wait(bSFull + 8 * buf, cG & 1u, abort_flag))) break;
        ++cG;
        tc_fence_after();
        // keys beyond the causal limit (and beyond the window, which the limit implies) do not exist
        const int nvalid = kb == it.qb ? r + 1 : DAM_TILE;
        const bool diag = kb == it.qb;
        uint4 words = make_uint4(0u, 0u, 0u, 0u);
        float tmax = -CUDART_INF_F, tsum = 0.f;
        uint32_t cur[32];
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          tmem_ld32(tS + c * 32, cur);
          tc_wait_ld();
          // raw dot products; the softmax scale (in log2 units) is applied inside the exponent's multiply-add
          float x[32];
#pragma unroll
          for (int q = 0; q < 32; ++q) x[q] = __uint_as_float(cur[q]);
          if (diag) {
#pragma unroll
            for (int q = 0; q < 32; ++q) x[q] = (c * 32 + q < nvalid) ? x[q] : -CUDART_INF_F;
          }
          if (!sweepB) {
            float c0 = -CUDART_INF_F, c1 = -CUDART_INF_F;
#pragma unroll
            for (int q = 0; q < 32; q += 4) { c0 = max3(c0, x[q], x[q + 1]); c1 = max3(c1, x[q + 2], x[q + 3]); }
            const float mn = fmaxf(tmax, fmaxf(c0, c1));          // maximum of the raw values (the scale is positive)
            if (mn > -CUDART_INF_F) {
              const float nm = -(mn * prm.scale_log2);
              float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
              for (int q = 0; q < 32; q += 4) {
                float y0, y1, y2, y3;
                fma2(y0, y1, x[q], x[q + 1], prm.scale_log2, prm.scale_log2, nm, nm);
                fma2(y2, y3, x[q + 2], x[q + 3], prm.scale_log2, prm.scale_log2, nm, nm);
                add2(a0, a1, a0, a1, ex2(y0), ex2(y1));
                add2(a2, a3, a2, a3, ex2(y2), ex2(y3));
              }
              tsum = tsum * ex2((tmax - mn) * prm.scale_log2) + ((a0 + a1) + (a2 + a3));     // tmax = -inf gives a factor 0
              tmax = mn;
            }
          } else if (Prow) {
            // the caller wants the map itself: every probability is computed and stored
            uint32_t word = 0u;
#pragma unroll
            for (int q = 0; q < 32; ++q) {
              const float p = ex2(fmaf(x[q], prm.scale_log2, -m)) * inv_l;    // -inf beyond the causal limit gives 0
              x[q] = p;
              word |= (p >= prm.pstar ? 1u : 0u) << q;
            }
            if (c == 0) words.x = word; else if (c == 1) words.y = word; else if (c == 2) words.z = word; else words.w = word;
            if (row_valid) {
              const int j0 = kb * DAM_TILE + c * 32;
#pragma unroll
              for (int q = 0; q < 32; ++q)
                if (j0 + q < L) Prow[j0 + q] = x[q];
            }
          } else {
            // only the decision p >= p* is needed.  p = 2^(x scale - m) / l, so an entry whose x scale - m lies
            // more than 2^-5 below log2(p* l) cannot reach p* (the margin is five orders of magnitude above the
            // rounding of the fast exponential and of the comparison on the raw value); groups of 8 columns with
            // no candidate in the whole warp skip the special-function unit.  Candidates are evaluated exactly
            // as in the branch above.
            uint32_t word = 0u;
#pragma unroll
            for (int q8 = 0; q8 < 32; q8 += 8) {
              bool any = false;
#pragma unroll
              for (int u = 0; u < 8; ++u) any |= x[q8 + u] > thr_raw;
              if (__any_sync(0xFFFFFFFFu, any)) {
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  const float p = ex2(fmaf(x[q8 + u], prm.scale_log2, -m)) * inv_l;
                  word |= (p >= prm.pstar ? 1u : 0u) << (q8 + u);
                }
              }
            }
            if (c == 0) words.x = word; else if (c == 1) words.y = word; else if (c == 2) words.z = word; else words.w = word;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bSEmpty + 8 * buf);
        if (!sweepB) {
          if (tmax > -CUDART_INF_F) {
            const float tm = tmax * prm.scale_log2;               // the tile's maximum in the scaled domain
            const float mn = fmaxf(m, tm);
            l = l * ex2(m - mn) + tsum * ex2(tm - mn);
            m = mn;
          }
        } else if (row_valid) {
          *reinterpret_cast<uint4*>(Mrow + kb * 4) = words;
        }
      }
      if (!ok) break;
      ++nitem;
      // zeros above the diagonal for the tiles this item does not visit: the true-mask words, and the map itself
      // when it is dumped
      if (row_valid && G == 0) {
        for (int kb = it.qb + 1; kb * 4 < W; ++kb) *reinterpret_cast<uint4*>(Mrow + kb * 4) = make_uint4(0u, 0u, 0u, 0u);
        if (Prow)
          for (int j = (it.qb + 1) * DAM_TILE; j < L; ++j) Prow[j] = 0.f;
      }
    }
  }

  if (*abort_flag && tid == 64) atomicMax(prm.status, (uint32_t)DAM_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

cudaError_t dam_launch_scores_sm100(const void* Q, const void* K, const dam_shape_t* s, const DamBuildCtx& c,
                                    float* dump, cudaStream_t st) {
  const int d = s->head_dim;
  if (s->dtype != DAM_BF16 || (d != 128 && d != 64)) return cudaErrorNotSupported;
  if (c.max_nL == 0) return cudaSuccess;
  int dev = 0;
  DamDeviceInfo di;
  cudaError_t e;
  if ((e = dam_current_device(&dev, &di)) != cudaSuccess) return e;
  if (di.cc_major != 10 || di.smem_optin < kSmemBytes) return cudaErrorNotSupported;
  if ((e = dam_device_table().once(dev, DAM_SETUP_SCORE_SMEM, [](void) -> cudaError_t {
         cudaError_t r = cudaFuncSetAttribute(score_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
         if (r != cudaSuccess) return r;
         return cudaFuncSetAttribute(score_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
       })) != cudaSuccess)
    return e;
  const int sm_count = di.sm_count;
  CUtensorMap tq, tk;
  if (!dam_make_tmap_bf16(&tq, Q, d, s->num_q_heads, s->total_tokens, s->q_stride_tok, s->q_stride_head) ||
      !dam_make_tmap_bf16(&tk, K, d, s->num_kv_heads, s->total_tokens, s->k_stride_tok, s->k_stride_head))
    return cudaErrorInvalidValue;
  ScoreParams p;
  p.blob = c.blob; p.dump = dump;
  p.status = reinterpret_cast<uint32_t*>(c.blob) + 1;
  p.work_counter = reinterpret_cast<uint32_t*>(c.scratch) + 2;
  // (the status block and the work counter at the start of the scratch buffer were cleared together with the
  // rule counters, before the blob was initialised: this kernel follows that one directly)
  p.num_seqs = c.num_seqs; p.Hq = c.Hq; p.group = c.Hq / c.Hkv; p.max_nL = c.max_nL;
  p.scale_log2 = c.scale * 1.4426950408889634f;
  p.pstar = c.pstar;
  const int items = c.max_nL * c.num_seqs * c.Hq;
  const int grid = items < sm_count ? items : sm_count;
  // launched as a programmatic dependent of the kernel that initialises the blob: its launch latency and its
  // prologue (barriers, TMEM, descriptors) hide under that kernel; it waits before it reads the blob
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (d == 128) return cudaLaunchKernelEx(&cfg, score_sm100_kernel<128>, tq, tk, p);
  return cudaLaunchKernelEx(&cfg, score_sm100_kernel<64>, tq, tk, p);
}
