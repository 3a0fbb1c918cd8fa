// Sparse flash attention on the 5th-generation tensor cores (sm_100a): bf16 inputs, head_dim 128.
//
// One persistent CTA per SM walks the work list of the mask blob (rows = (head, 128-row query block),
// longest tile list first).  Warp roles:
//   warp 0      TMA producer: Q tile once per row, then the K / V tiles of the listed kv tiles into a
//               ring of 32 KB shared-memory slots (128-byte swizzle, two 64-column boxes per tile);
//   warp 1      MMA issuer (one elected thread): S = Q K^T into one of two TMEM buffers, then
//               O += P V with P read from TMEM; completion is signalled with tcgen05.commit;
//   warps 2-5   softmax: one thread per query row reads its S row from TMEM, applies the tile's mask
//               bits where the tile is not fully active, keeps the running max / sum, writes P (bf16)
//               back to TMEM, rescales O in TMEM when the running max moved by more than 2^8, and
//               finally normalises and stores O and the log-sum-exp.
// Only the tiles the mask lists are ever loaded or multiplied (paper Sec. 4.3: masked logits are -inf).
// Every wait is bounded; an expired wait sets the status word in the scratch buffer and the CTA
// drains and exits.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "dam_internal.cuh"
#include "sm100_ptx.cuh"

using namespace sm100;

namespace {

constexpr int kSlots = 6;
constexpr int kSlotBytes = 32768;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;      // S buffers at columns 0 and 128
constexpr uint32_t kColO = 256;    // O accumulator
constexpr uint32_t kColP = 384;    // P buffers (bf16 pairs) at columns 384 and 448
constexpr float kRescaleThreshold = 8.0f;

struct SmemLayout {
  static constexpr int q = 0;
  static constexpr int slots = kSlotBytes;
  static constexpr int bars = kSlotBytes * (1 + kSlots);
  // barriers (8 bytes each): q_full, q_empty, slot_full[kSlots], slot_empty[kSlots], s_full[2], p_full[2], pv_done
  static constexpr int n_bars = 2 + 2 * kSlots + 2 + 2 + 1;
  static constexpr int tmem_slot = bars + 8 * n_bars;
  static constexpr int abort_flag = tmem_slot + 4;
  static constexpr int total = abort_flag + 4;
};
constexpr int kSmemBytes = SmemLayout::total + 1024;   // + slack for the 1024-byte alignment

struct AttnParams {
  const unsigned char* blob;
  __nv_bfloat16* O;
  float* lse;
  uint32_t* status;         // scratch status word
  int Hq, group, total_tokens, causal;
  int64_t o_stride_tok, o_stride_head;
  float scale_log2;         // softmax scale * log2(e)
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct Item {
  int head, seq_tok0, qb, S;
  uint32_t t0, nt;
};

__device__ __forceinline__ Item load_item(const unsigned char* blob, const DamHeader* H, int w, DamSeq* sq_out) {
  const uint32_t row = __ldg(reinterpret_cast<const uint32_t*>(blob + H->off_work) + w);
  const int h = row / H->total_qblocks, gqb = row % H->total_qblocks;
  const int b = __ldg(reinterpret_cast<const int32_t*>(blob + H->off_qbseq) + gqb);
  const DamSeq sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[b];
  const uint32_t* tp = reinterpret_cast<const uint32_t*>(blob + H->off_tile_ptr);
  Item it;
  it.head = h; it.seq_tok0 = sq.tok_start; it.qb = gqb - sq.first_qblock; it.S = sq.S;
  it.t0 = __ldg(tp + row); it.nt = __ldg(tp + row + 1) - it.t0;
  if (sq_out) *sq_out = sq;
  return it;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const AttnParams prm) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sQ = sbase + SmemLayout::q;
  const uint32_t sSlots = sbase + SmemLayout::slots;
  const uint32_t bar0 = sbase + SmemLayout::bars;
  const uint32_t bQFull = bar0, bQEmpty = bar0 + 8;
  const uint32_t bSlotFull = bar0 + 16, bSlotEmpty = bSlotFull + 8 * kSlots;
  const uint32_t bSFull = bSlotEmpty + 8 * kSlots, bPFull = bSFull + 16, bPvDone = bPFull + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + SmemLayout::tmem_slot);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + SmemLayout::abort_flag);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const unsigned char* blob = prm.blob;
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int nrows = H->rows;
  const uint32_t* tiles = reinterpret_cast<const uint32_t*>(blob + H->off_tiles);

  if (tid == 0) {
    mbar_init(bQFull, 1); mbar_init(bQEmpty, 1);
    for (int s = 0; s < kSlots; ++s) { mbar_init(bSlotFull + 8 * s, 1); mbar_init(bSlotEmpty + 8 * s, 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(bSFull + 8 * s, 1); mbar_init(bPFull + 8 * s, 128); }
    mbar_init(bPvDone, 1);
    *abort_flag = 0u;
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 0) { tmem_alloc(smem_u32(tmem_slot), kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t sc = 0, ic = 0;
      uint32_t armed[kSlots];
#pragma unroll
      for (int s = 0; s < kSlots; ++s) armed[s] = 2u;      // 2 = never armed
      bool ok = true;
      auto load_tile = [&](const CUtensorMap* tm, int head, int tok) -> bool {
        const uint32_t s = sc % kSlots, ph = (sc / kSlots) & 1u;
        if (!mbar_wait(bSlotEmpty + 8 * s, ph ^ 1u, abort_flag)) return false;
        const uint32_t dst = sSlots + s * kSlotBytes, bar = bSlotFull + 8 * s;
        mbar_arrive_expect_tx(bar, kSlotBytes);
        tma_load_3d(dst, tm, bar, 0, head, tok);
        tma_load_3d(dst + 16384, tm, bar, 64, head, tok);
        armed[s] = ph;
        ++sc;
        return true;
      };
      for (int w = blockIdx.x; w < nrows && ok; w += gridDim.x) {
        const Item it = load_item(blob, H, w, nullptr);
        if (it.nt == 0) continue;
        if (!(ok = mbar_wait(bQEmpty, (ic & 1u) ^ 1u, abort_flag))) break;
        mbar_arrive_expect_tx(bQFull, kSlotBytes);
        tma_load_3d(sQ, &tmQ, bQFull, 0, it.head, it.seq_tok0 + it.qb * DAM_TILE);
        tma_load_3d(sQ + 16384, &tmQ, bQFull, 64, it.head, it.seq_tok0 + it.qb * DAM_TILE);
        ++ic;
        const int kvh = it.head / prm.group;
        // ring order = order in which the MMA warp consumes: K0, K1, V0, K2, V1, ..., V(n-1)
        for (uint32_t t = 0; t < it.nt && ok; ++t) {
          const int kb = (int)(__ldg(tiles + it.t0 + t) & 0x0FFFFFFFu);
          ok = load_tile(&tmK, kvh, it.seq_tok0 + kb * DAM_TILE);
          if (ok && t >= 1) {
            const int kbp = (int)(__ldg(tiles + it.t0 + t - 1) & 0x0FFFFFFFu);
            ok = load_tile(&tmV, kvh, it.seq_tok0 + kbp * DAM_TILE);
          }
        }
        if (ok) {
          const int kbl = (int)(__ldg(tiles + it.t0 + it.nt - 1) & 0x0FFFFFFFu);
          ok = load_tile(&tmV, kvh, it.seq_tok0 + kbl * DAM_TILE);
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
      const uint32_t idesc_pv = idesc_bf16_f32(128, 128, 1);
      uint32_t sc = 0, ic = 0, g = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < nrows && ok; w += gridDim.x) {
        const Item it = load_item(blob, H, w, nullptr);
        if (it.nt == 0) continue;
        if (!(ok = mbar_wait(bQFull, ic & 1u, abort_flag))) break;
        ++ic;
        tc_fence_after();
        auto do_pv = [&](uint32_t u) -> bool {
          const uint32_t gt = g + u, buf = gt & 1u;
          if (!mbar_wait(bPFull + 8 * buf, (gt >> 1) & 1u, abort_flag)) return false;
          const uint32_t s = sc % kSlots;
          if (!mbar_wait(bSlotFull + 8 * s, (sc / kSlots) & 1u, abort_flag)) return false;
          tc_fence_after();
          const uint32_t vaddr = sSlots + s * kSlotBytes;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            // V is MN-major: 16 keys per step = 2048 bytes; 64-column halves 16384 bytes apart
            const uint64_t bdesc = smem_desc_sw128(vaddr + ks * 2048, 16384, 1024);
            mma_ts(tmem + kColO, tmem + kColP + buf * 64 + ks * 8, bdesc, idesc_pv, (u > 0 || ks > 0) ? 1u : 0u);
          }
          tc_commit(bSlotEmpty + 8 * s);
          tc_commit(bPvDone);
          ++sc;
          return true;
        };
        for (uint32_t t = 0; t < it.nt && ok; ++t) {
          const uint32_t gt = g + t, buf = gt & 1u;
          const uint32_t s = sc % kSlots;
          if (!(ok = mbar_wait(bSlotFull + 8 * s, (sc / kSlots) & 1u, abort_flag))) break;
          tc_fence_after();
          const uint32_t kaddr = sSlots + s * kSlotBytes;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
            const uint64_t adesc = smem_desc_sw128(sQ + off, 16, 1024);
            const uint64_t bdesc = smem_desc_sw128(kaddr + off, 16, 1024);
            mma_ss(tmem + kColS + buf * 128, adesc, bdesc, idesc_qk, ks > 0 ? 1u : 0u);
          }
          tc_commit(bSlotEmpty + 8 * s);
          tc_commit(bSFull + 8 * buf);
          if (t + 1 == it.nt) tc_commit(bQEmpty);
          ++sc;
          if (t >= 1) ok = do_pv(t - 1);
        }
        if (ok) ok = do_pv(it.nt - 1);
        g += it.nt;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax / epilogue warps
    const int r = (warp & 3) * 32 + lane;                    // row of the tile = TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    uint32_t g = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < nrows && ok; w += gridDim.x) {
      DamSeq sq;
      const Item it = load_item(blob, H, w, &sq);
      const int i = it.qb * DAM_TILE + r;
      const bool row_valid = i < it.S;
      __nv_bfloat16* orow = prm.O + (int64_t)(it.seq_tok0 + i) * prm.o_stride_tok + (int64_t)it.head * prm.o_stride_head;
      float* lse_p = prm.lse + (int64_t)it.head * prm.total_tokens + it.seq_tok0 + i;
      if (it.nt == 0) {
        if (row_valid) {
          const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
          for (int c = 0; c < 16; ++c) reinterpret_cast<uint4*>(orow)[c] = z;
          *lse_p = -CUDART_INF_F;
        }
        continue;
      }
      const DamHeadBits hb = dam_head_bits(blob, H, sq, it.head);
      float m_ref = -CUDART_INF_F;   // reference max (scaled, log2 domain) that P and O are expressed against
      float l = 0.f;
      for (uint32_t t = 0; t < it.nt; ++t) {
        const uint32_t e = __ldg(tiles + it.t0 + t);
        const int kb = (int)(e & 0x0FFFFFFFu);
        const uint32_t kind = e >> 28;
        const bool need_mask = (kind != DAM_KIND_FULL) || (prm.causal && kb >= it.qb) || ((kb + 1) * DAM_TILE > it.S);
        uint4 bits = make_uint4(~0u, ~0u, ~0u, ~0u);
        if (need_mask) bits = dam_apply_bits(hb, kind, i, kb, prm.causal);
        const uint32_t gt = g + t, buf = gt & 1u;
        if (!(ok = mbar_wait(bSFull + 8 * buf, (gt >> 1) & 1u, abort_flag))) break;
        tc_fence_after();
        // ---- S row -> registers (raw dot products), masked entries -> -inf
        float x[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t rr[32];
          tmem_ld32(tmem + lane_addr + kColS + buf * 128 + c * 32, rr);
          tc_wait_ld();
          const uint32_t word = c == 0 ? bits.x : (c == 1 ? bits.y : (c == 2 ? bits.z : bits.w));
#pragma unroll
          for (int q = 0; q < 32; ++q) {
            float v = __uint_as_float(rr[q]);
            if (need_mask) v = ((word >> q) & 1u) ? v : -CUDART_INF_F;
            x[c * 32 + q] = v;
          }
        }
        float mx = -CUDART_INF_F;
#pragma unroll
        for (int q = 0; q < 128; ++q) mx = fmaxf(mx, x[q]);
        const float m_new = fmaxf(m_ref, mx * prm.scale_log2);
        // move the reference only when it is the first tile or the max grew by more than the threshold
        bool move = (t == 0) || (m_new - m_ref > kRescaleThreshold);   // -inf reference: inf > 8 is true
        if (m_new == -CUDART_INF_F) move = false;
        float alpha = 1.f;
        if (move) {
          alpha = (m_ref == -CUDART_INF_F) ? 0.f : ex2(m_ref - m_new);
          m_ref = m_new;
        }
        const float mm = (m_ref == -CUDART_INF_F) ? 0.f : m_ref;
        float sum = 0.f;
        uint32_t pk[64];
#pragma unroll
        for (int q = 0; q < 64; ++q) {
          const float p0 = ex2(fmaf(x[2 * q], prm.scale_log2, -mm));
          const float p1 = ex2(fmaf(x[2 * q + 1], prm.scale_log2, -mm));
          sum += p0 + p1;
          __nv_bfloat162 hpair = __floats2bfloat162_rn(p0, p1);
          pk[q] = *reinterpret_cast<uint32_t*>(&hpair);
        }
        l = l * alpha + sum;
        tmem_st32(tmem + lane_addr + kColP + buf * 64, pk);
        tmem_st32(tmem + lane_addr + kColP + buf * 64 + 32, pk + 32);
        // ---- O must be complete up to the previous tile before it is rescaled / before P(t) is consumed
        if (t > 0) {
          if (!(ok = mbar_wait(bPvDone, (gt - 1u) & 1u, abort_flag))) break;
          tc_fence_after();
          const bool resc = alpha != 1.f;
          if (__any_sync(0xFFFFFFFFu, resc)) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t rr[32];
              tmem_ld32(tmem + lane_addr + kColO + c * 32, rr);
              tc_wait_ld();
#pragma unroll
              for (int q = 0; q < 32; ++q) rr[q] = __float_as_uint(__uint_as_float(rr[q]) * alpha);
              tmem_st32(tmem + lane_addr + kColO + c * 32, rr);
            }
          }
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bPFull + 8 * buf);
      }
      if (!ok) break;
      // ---- epilogue: O / l and the log-sum-exp
      const uint32_t glast = g + it.nt - 1u;
      if (!(ok = mbar_wait(bPvDone, glast & 1u, abort_flag))) break;
      tc_fence_after();
      const float inv = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t rr[32];
        tmem_ld32(tmem + lane_addr + kColO + c * 32, rr);
        tc_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int v4 = 0; v4 < 4; ++v4) {
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              float a = l > 0.f ? __uint_as_float(rr[v4 * 8 + 2 * q]) * inv : 0.f;
              float b = l > 0.f ? __uint_as_float(rr[v4 * 8 + 2 * q + 1]) * inv : 0.f;
              __nv_bfloat162 hpair = __floats2bfloat162_rn(a, b);
              o[q] = *reinterpret_cast<uint32_t*>(&hpair);
            }
            reinterpret_cast<uint4*>(orow)[c * 4 + v4] = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
      }
      if (row_valid) *lse_p = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -CUDART_INF_F;
      tc_fence_before();
      g += it.nt;
    }
  }

  if (*abort_flag && tid == 64) atomicMax(prm.status, (uint32_t)DAM_ERR_DEVICE_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

cudaError_t dam_launch_attn_sm100(const void* Q, const void* K, const void* V, const void* blob,
                                  const dam_shape_t* s, int causal, float scale, void* O, float* lse, void* scratch,
                                  cudaStream_t st) {
  if (s->dtype != DAM_BF16 || s->head_dim != 128) return cudaErrorNotSupported;
  if (s->total_tokens == 0) return cudaSuccess;
  static int sm_count = 0, smem_optin = 0;
  if (sm_count == 0) {
    int dev = 0;
    cudaError_t e;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    int cc_major = 0;
    cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev);
    if (cc_major != 10) return cudaErrorNotSupported;
    cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (smem_optin < kSmemBytes) return cudaErrorNotSupported;
    if ((e = cudaFuncSetAttribute(attn_sm100_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess)
      return e;
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  CUtensorMap tq, tk, tv;
  if (!dam_make_tmap_bf16(&tq, Q, 128, s->num_q_heads, s->total_tokens, s->q_stride_tok, s->q_stride_head) ||
      !dam_make_tmap_bf16(&tk, K, 128, s->num_kv_heads, s->total_tokens, s->k_stride_tok, s->k_stride_head) ||
      !dam_make_tmap_bf16(&tv, V, 128, s->num_kv_heads, s->total_tokens, s->v_stride_tok, s->v_stride_head))
    return cudaErrorInvalidValue;
  int rows = 0;
  for (int b = 0; b < s->num_seqs; ++b)
    rows += (s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b] + DAM_TILE - 1) / DAM_TILE;
  rows *= s->num_q_heads;
  if (rows == 0) return cudaSuccess;
  AttnParams p;
  p.blob = reinterpret_cast<const unsigned char*>(blob);
  p.O = reinterpret_cast<__nv_bfloat16*>(O);
  p.lse = lse;
  p.status = reinterpret_cast<uint32_t*>(scratch) + 1;
  p.Hq = s->num_q_heads; p.group = s->num_q_heads / s->num_kv_heads; p.total_tokens = s->total_tokens;
  p.causal = causal;
  p.o_stride_tok = s->o_stride_tok; p.o_stride_head = s->o_stride_head;
  p.scale_log2 = scale * 1.4426950408889634f;
  const int grid = rows < sm_count ? rows : sm_count;
  attn_sm100_kernel<<<grid, kThreads, kSmemBytes, st>>>(tq, tk, tv, p);
  return cudaGetLastError();
}
