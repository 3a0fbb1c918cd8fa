// Plain CUDA-core kernels (fp32 arithmetic, any head_dim that is a multiple of 8 up to 256, bf16
// or fp32 inputs).  They serve the fp32 configuration and every shape the tensor-core kernels do
// not cover, and are the on-device cross-check for those kernels.  One warp per query row.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "dam_internal.cuh"

namespace {

template <typename T> struct Ld8;
template <> struct Ld8<float> {
  static __device__ __forceinline__ void load(const float* p, float* o) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p));
    float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
  }
  static __device__ __forceinline__ float one(const float* p) { return __ldg(p); }
  static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
};
template <> struct Ld8<__nv_bfloat16> {
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* o) {
    uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      o[2 * q] = __uint_as_float(w[q] << 16);
      o[2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
    }
  }
  static __device__ __forceinline__ float one(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

template <typename T>
__device__ __forceinline__ float dot_row(const float* __restrict__ q_s, const T* __restrict__ k, int d) {
  float acc = 0.f;
  for (int t = 0; t < d; t += 8) {
    float kv[8];
    Ld8<T>::load(k + t, kv);
#pragma unroll
    for (int u = 0; u < 8; ++u) acc = fmaf(q_s[t + u], kv[u], acc);
  }
  return acc;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

// ---------------------------------------------------------------------------------------------
// Window scores: causal softmax over the first L tokens, then the single-compare threshold.
// Two sweeps over the keys of a row (max / sum, then probabilities); the fp32 probability that is
// compared with p* is the very value written to the dump.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void scores_ref_kernel(unsigned char* blob, const T* __restrict__ Q, const T* __restrict__ K,
                                  int Hq, int group, int d, int64_t qst, int64_t qsh, int64_t kst, int64_t ksh,
                                  float scale, float pstar, float* __restrict__ dump) {
  extern __shared__ float smem[];
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int sh = blockIdx.y;
  const int b = sh / Hq, h = sh % Hq;
  const DamSeq sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[b];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int i = blockIdx.x * nw + warp;
  if (i >= sq.L) return;
  float* q_s = smem + warp * d;
  const T* qrow = Q + (int64_t)(sq.tok_start + i) * qst + (int64_t)h * qsh;
  for (int t = lane; t < d; t += 32) q_s[t] = Ld8<T>::one(qrow + t);
  __syncwarp();
  const T* Kh = K + (int64_t)sq.tok_start * kst + (int64_t)(h / group) * ksh;
  float m = -CUDART_INF_F, l = 0.f;
  for (int j = lane; j <= i; j += 32) {
    float s = dot_row<T>(q_s, Kh + (int64_t)j * kst, d) * scale;
    float mn = fmaxf(m, s);
    l = l * expf(m - mn) + expf(s - mn);
    m = mn;
  }
  float mw = warp_max(m);
  l = (m == -CUDART_INF_F) ? 0.f : l * expf(m - mw);
  l = warp_sum(l);
  uint32_t* M = reinterpret_cast<uint32_t*>(blob + H->off_true) + sq.true_off + (uint64_t)h * sq.L * sq.W;
  float* Ph = dump ? dump + sq.p_off + (uint64_t)h * sq.L * sq.L + (uint64_t)i * sq.L : nullptr;
  for (int w = 0; w < sq.W; ++w) {
    int j = w * 32 + lane;
    float p = 0.f;
    if (j <= i) {
      float s = dot_row<T>(q_s, Kh + (int64_t)j * kst, d) * scale;
      p = expf(s - mw) / l;
    }
    if (Ph && j < sq.L) Ph[j] = p;
    uint32_t word = __ballot_sync(0xFFFFFFFFu, p >= pstar);
    if (lane == 0) M[(size_t)i * sq.W + w] = word;
  }
}

// ---------------------------------------------------------------------------------------------
// Masked attention over the listed tiles.  Block = 4 warps = one (head, q-block) row of the tile
// list; each warp walks 32 of its 128 query rows.  Online softmax in fp32.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void attn_ref_kernel(const unsigned char* blob, const T* __restrict__ Q, const T* __restrict__ K,
                                const T* __restrict__ V, int Hq, int group, int d, int64_t qst, int64_t qsh,
                                int64_t kst, int64_t ksh, int64_t vst, int64_t vsh, int64_t ost, int64_t osh,
                                int causal, float scale, T* __restrict__ O, float* __restrict__ lse, int total_tokens,
                                const int32_t* __restrict__ ranges) {
  extern __shared__ float smem[];
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int row = blockIdx.x;
  const int h = row / H->total_qblocks, gqb = row % H->total_qblocks;
  const int b = reinterpret_cast<const int32_t*>(blob + H->off_qbseq)[gqb];
  const DamSeq sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[b];
  const int qb = gqb - sq.first_qblock;
  if (ranges) {                                 // row ranges: whole pairs of query blocks, chosen by the pair's first row
    const int r0 = (qb & ~1) * DAM_TILE;
    if (r0 < ranges[2 * b] || r0 >= ranges[2 * b + 1]) return;
  }
  const uint32_t* tile_ptr = reinterpret_cast<const uint32_t*>(blob + H->off_tile_ptr);
  const uint32_t* tiles = reinterpret_cast<const uint32_t*>(blob + H->off_tiles);
  const uint32_t t0 = tile_ptr[row], t1 = tile_ptr[row + 1];
  const DamHeadBits hb = dam_head_bits(blob, H, sq, h);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  float* q_s = smem + warp * d;
  const T* Kh = K + (int64_t)sq.tok_start * kst + (int64_t)(h / group) * ksh;
  const T* Vh = V + (int64_t)sq.tok_start * vst + (int64_t)(h / group) * vsh;
  const int nd = d / 32 + ((d % 32) ? 1 : 0);

  for (int r = warp; r < DAM_TILE; r += nw) {
    const int i = qb * DAM_TILE + r;
    if (i >= sq.S) break;
    const T* qrow = Q + (int64_t)(sq.tok_start + i) * qst + (int64_t)h * qsh;
    __syncwarp();
    for (int t = lane; t < d; t += 32) q_s[t] = Ld8<T>::one(qrow + t);
    __syncwarp();
    float acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc[u] = 0.f;
    float m = -CUDART_INF_F, l = 0.f;
    for (uint32_t t = t0; t < t1; ++t) {
      const uint32_t e = __ldg(tiles + t);
      if ((e >> 28) == 0u) continue;                    // padding behind the row's entries
      const int kb = (int)(e & 0x0FFFFFFFu);
      const uint4 bits = dam_apply_bits(hb, e >> 28, i, kb, causal);
      const uint32_t w4[4] = {bits.x, bits.y, bits.z, bits.w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t word = w4[c];
        if (!word) continue;
        const int jb = kb * DAM_TILE + c * 32;
        const bool act = (word >> lane) & 1u;
        float s = -CUDART_INF_F;
        if (act) s = dot_row<T>(q_s, Kh + (int64_t)(jb + lane) * kst, d) * scale;
        float mn = fmaxf(m, warp_max(s));
        float corr = (m == -CUDART_INF_F) ? 0.f : expf(m - mn);
        float p = act ? expf(s - mn) : 0.f;
        l = l * corr + warp_sum(p);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc[u] *= corr;
        m = mn;
        while (word) {
          int kk = __ffs(word) - 1;
          word &= word - 1;
          float pj = __shfl_sync(0xFFFFFFFFu, p, kk);
          const T* vrow = Vh + (int64_t)(jb + kk) * vst;
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            int t_ = lane + 32 * u;
            if (u < nd && t_ < d) acc[u] = fmaf(pj, Ld8<T>::one(vrow + t_), acc[u]);
          }
        }
      }
    }
    T* orow = O + (int64_t)(sq.tok_start + i) * ost + (int64_t)h * osh;
    const float inv = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      int t_ = lane + 32 * u;
      if (u < nd && t_ < d) Ld8<T>::store(orow + t_, acc[u] * inv);
    }
    if (lane == 0) lse[(int64_t)h * total_tokens + sq.tok_start + i] = l > 0.f ? m + logf(l) : -CUDART_INF_F;
  }
}

}  // namespace

cudaError_t dam_launch_scores_ref(const void* Q, const void* K, const dam_shape_t* s, const DamBuildCtx& c,
                                  float* dump, cudaStream_t st) {
  if (c.max_L == 0) return cudaSuccess;
  const int nw = 8;
  dim3 grid((c.max_L + nw - 1) / nw, c.num_seqs * c.Hq);
  size_t sm = (size_t)nw * c.d * sizeof(float);
  int group = c.Hq / c.Hkv;
  if (c.dtype == DAM_F32)
    scores_ref_kernel<float><<<grid, nw * 32, sm, st>>>(c.blob, (const float*)Q, (const float*)K, c.Hq, group, c.d,
                                                        s->q_stride_tok, s->q_stride_head, s->k_stride_tok,
                                                        s->k_stride_head, c.scale, c.pstar, dump);
  else
    scores_ref_kernel<__nv_bfloat16><<<grid, nw * 32, sm, st>>>(c.blob, (const __nv_bfloat16*)Q,
                                                                (const __nv_bfloat16*)K, c.Hq, group, c.d,
                                                                s->q_stride_tok, s->q_stride_head, s->k_stride_tok,
                                                                s->k_stride_head, c.scale, c.pstar, dump);
  return cudaGetLastError();
}

cudaError_t dam_launch_attn_ref(const void* Q, const void* K, const void* V, const void* blob, const dam_shape_t* s,
                                int causal, float scale, void* O, float* lse, void* scratch, const int32_t* ranges,
                                cudaStream_t st) {
  (void)scratch;
  int rows = 0;
  for (int b = 0; b < s->num_seqs; ++b)
    rows += (s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b] + DAM_TILE - 1) / DAM_TILE;
  rows *= s->num_q_heads;
  if (rows == 0) return cudaSuccess;
  const int nw = 4;
  size_t sm = (size_t)nw * s->head_dim * sizeof(float);
  int group = s->num_q_heads / s->num_kv_heads;
  if (s->dtype == DAM_F32)
    attn_ref_kernel<float><<<rows, nw * 32, sm, st>>>((const unsigned char*)blob, (const float*)Q, (const float*)K,
        (const float*)V, s->num_q_heads, group, s->head_dim, s->q_stride_tok, s->q_stride_head, s->k_stride_tok,
        s->k_stride_head, s->v_stride_tok, s->v_stride_head, s->o_stride_tok, s->o_stride_head, causal, scale,
        (float*)O, lse, s->total_tokens, ranges);
  else
    attn_ref_kernel<__nv_bfloat16><<<rows, nw * 32, sm, st>>>((const unsigned char*)blob, (const __nv_bfloat16*)Q,
        (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, s->num_q_heads, group, s->head_dim, s->q_stride_tok,
        s->q_stride_head, s->k_stride_tok, s->k_stride_head, s->v_stride_tok, s->v_stride_head, s->o_stride_tok,
        s->o_stride_head, causal, scale, (__nv_bfloat16*)O, lse, s->total_tokens, ranges);
  return cudaGetLastError();
}
