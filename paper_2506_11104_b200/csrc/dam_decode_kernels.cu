// Generation-time attention under the stored patterns (paper Sec. 4.3 applied to one new token per sequence).
//
// A query at position i of a sequence attends, among the keys 0..i of the KV cache, to the keys the extended
// mask keeps for row i: inside the window (i < L) the row of the true mask; below it the matched columns c
// (V[c] = 1) and, for every matched diagonal r (D[r] = 1), the key i - r.  Nothing else of the blob is used (no
// tile lists), so i may lie beyond the length the blob was built for.  The work is a gather of a few hundred K
// and V rows per (sequence, head): bound by memory latency and bandwidth, not by arithmetic, so it runs on the
// CUDA cores: one block of 8 warps per (sequence, query head).  The block expands the pattern words into a key
// list in shared memory (a thread per word, block-wide prefix sum), then the keys are dealt to the warps: 8
// lanes share one key (each holds head_dim / 8 dimensions of q and of the output), every lane group has the
// K and V rows of 4 keys in flight (16 keys per warp), online softmax in the log2 domain, partial results
// merged through shuffles and shared memory.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "dam_internal.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kKeysPerGroup = 2;               // keys a lane group has in flight per step
constexpr int kBlocksPerSM = 4;                // resident blocks the register limit is sized for
constexpr int kRoundWords = 256;               // pattern words the block expands at a time (<= 8192 keys, 32 KB)

template <typename T, int N> struct LdN;       // N consecutive elements -> float
template <int N> struct LdN<float, N> {
  static __device__ __forceinline__ void load(const float* p, float* o) {
#pragma unroll
    for (int t = 0; t < N; t += 4) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(p + t));
      o[t] = a.x; o[t + 1] = a.y; o[t + 2] = a.z; o[t + 3] = a.w;
    }
  }
};
template <int N> struct LdN<__nv_bfloat16, N> {
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* o) {
#pragma unroll
    for (int t = 0; t < N; t += 8) {
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(p + t));
      const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        o[t + 2 * q] = __uint_as_float(w[q] << 16);
        o[t + 2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
      }
    }
  }
};
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Running softmax state of one lane group: max m (log2 domain), sum l, DPL output dimensions.
template <int DPL>
struct Acc {
  float m, l, o[DPL];
  __device__ __forceinline__ void init() {
    m = -CUDART_INF_F; l = 0.f;
#pragma unroll
    for (int t = 0; t < DPL; ++t) o[t] = 0.f;
  }
  // state of another lane (same dimensions, other keys) fetched with a shuffle
  __device__ __forceinline__ void merge_xor(int mask) {
    const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m, mask);
    const float l2 = __shfl_xor_sync(0xFFFFFFFFu, l, mask);
    const float mn = fmaxf(m, m2);
    const float a = (m == -CUDART_INF_F) ? 0.f : fast_ex2(m - mn);
    const float b = (m2 == -CUDART_INF_F) ? 0.f : fast_ex2(m2 - mn);
    l = l * a + l2 * b;
#pragma unroll
    for (int t = 0; t < DPL; ++t) {
      const float o2 = __shfl_xor_sync(0xFFFFFFFFu, o[t], mask);
      o[t] = o[t] * a + o2 * b;
    }
    m = mn;
  }
};

// Raw (unconverted) loads of N consecutive elements, so that many rows can be in flight per lane.
template <typename T, int N> struct Raw;
template <int N> struct Raw<float, N> {
  float4 v[N / 4];
  __device__ __forceinline__ void load(const float* p) {
#pragma unroll
    for (int t = 0; t < N / 4; ++t) v[t] = __ldg(reinterpret_cast<const float4*>(p) + t);
  }
  __device__ __forceinline__ void to_float(float* o) const {
#pragma unroll
    for (int t = 0; t < N / 4; ++t) { o[4 * t] = v[t].x; o[4 * t + 1] = v[t].y; o[4 * t + 2] = v[t].z; o[4 * t + 3] = v[t].w; }
  }
};
template <int N> struct Raw<__nv_bfloat16, N> {
  uint4 v[N / 8];
  __device__ __forceinline__ void load(const __nv_bfloat16* p) {
#pragma unroll
    for (int t = 0; t < N / 8; ++t) v[t] = __ldg(reinterpret_cast<const uint4*>(p) + t);
  }
  __device__ __forceinline__ void to_float(float* o) const {
#pragma unroll
    for (int t = 0; t < N / 8; ++t) {
      const uint32_t w[4] = {v[t].x, v[t].y, v[t].z, v[t].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        o[8 * t + 2 * q] = __uint_as_float(w[q] << 16);
        o[8 * t + 2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
      }
    }
  }
};

template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32, kBlocksPerSM)
decode_kernel(const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
              const unsigned char* __restrict__ blob, const int32_t* __restrict__ cu, const int32_t* __restrict__ pos_dev,
              int num_seqs, int Hq, int group, int64_t kst, int64_t ksh, int64_t vst, int64_t vsh, float scale_log2,
              T* __restrict__ O, float* __restrict__ lse, uint32_t* status) {
  constexpr int DPL = D / 8;
  constexpr int kThreads = kWarps * 32;
  __shared__ int keys[kRoundWords * 32];
  __shared__ int warp_tot[kWarps];
  __shared__ float sm_m[kWarps], sm_l[kWarps];
  __shared__ float sm_o[kWarps][D];
  const int h = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 3, sub = lane & 7;
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  T* orow = O + ((int64_t)b * Hq + h) * D;
  float* lse_p = lse + (int64_t)b * Hq + h;
  bool bad = H->magic != DAM_MAGIC || H->num_seqs != num_seqs || H->num_q_heads != Hq;
  int pos = 0, cap = 0;
  if (!bad) {
    pos = pos_dev[b];
    cap = cu[b + 1] - cu[b];
    bad = pos < 0 || pos >= cap;
  }
  if (bad) {
    if (tid == 0) { atomicMax(status, (uint32_t)DAM_ERR_INVALID_ARGUMENT); *lse_p = -CUDART_INF_F; }
    for (int t = tid; t < D; t += blockDim.x) orow[t] = from_float<T>(0.f);
    return;
  }
  const DamSeq sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[b];
  const DamHeadBits hb = dam_head_bits(blob, H, sq, h);
  const int L = hb.L, W = hb.W;
  const bool in_window = pos < L;
  // index space of pattern words: [0, W) the row of the true mask (inside the window) or the matched columns;
  // [W, 2W) the matched diagonals (below the window only)
  const int nwords = in_window ? W : 2 * W;
  const T* Kb = K + (int64_t)cu[b] * kst + (int64_t)(h / group) * ksh + sub * DPL;
  const T* Vb = V + (int64_t)cu[b] * vst + (int64_t)(h / group) * vsh + sub * DPL;
  float qf[DPL];
  LdN<T, DPL>::load(q + ((int64_t)b * Hq + h) * D + sub * DPL, qf);
#pragma unroll
  for (int t = 0; t < DPL; ++t) qf[t] *= scale_log2;
  Acc<DPL> acc;
  acc.init();
  for (int w0 = 0; w0 < nwords; w0 += kRoundWords) {
    // ---- the block expands up to kRoundWords pattern words into one key list (a thread per word)
    const int nw = min(kRoundWords, nwords - w0);
    int total = 0;
    __syncthreads();                                          // the previous round's list is no longer read
    for (int wb = 0; wb < nw; wb += kThreads) {
      const int wi = w0 + wb + tid;
      uint32_t word = 0u;
      if (wb + tid < nw) {
        if (in_window) {
          word = __ldg(hb.M + (size_t)pos * W + wi);
        } else if (wi < W) {
          word = __ldg(hb.V + wi);
        } else {
          // diagonal r = 32 (wi - W) + k selects key pos - r; drop it when that key is a matched column (it
          // is already in the list): bit k of the reversed 32-bit window of V that ends at key pos - 32 (wi - W)
          const int r0 = 32 * (wi - W);
          word = __ldg(hb.D + (wi - W)) & ~__brev(dam_window32(hb.V, W, pos - r0 - 31));
        }
      }
      const int cnt = __popc(word);
      int off = cnt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xFFFFFFFFu, off, o);
        if (lane >= o) off += y;
      }
      if (lane == 31) warp_tot[warp] = off;
      __syncthreads();
      int before = total;
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const int wt = warp_tot[w];
        if (w < warp) before += wt;
        total += wt;
      }
      off += before - cnt;
      while (word) {
        const int k = __ffs(word) - 1;
        word &= word - 1u;
        keys[off++] = (in_window || wi < W) ? 32 * wi + k : pos - (32 * (wi - W) + k);
      }
      __syncthreads();
    }
    // ---- every lane group takes kKeysPerGroup keys per step; the K and V rows of all of them are requested
    //      before any is used
    for (int base = warp * (4 * kKeysPerGroup); base < total; base += kWarps * 4 * kKeysPerGroup) {
      Raw<T, DPL> kr[kKeysPerGroup], vr[kKeysPerGroup];
      bool valid[kKeysPerGroup];
#pragma unroll
      for (int u = 0; u < kKeysPerGroup; ++u) {
        const int idx = base + u * 4 + g;
        valid[u] = idx < total;
        const int j = valid[u] ? keys[idx] : 0;
        kr[u].load(Kb + (int64_t)j * kst);
        vr[u].load(Vb + (int64_t)j * vst);
      }
      float sc[kKeysPerGroup];
#pragma unroll
      for (int u = 0; u < kKeysPerGroup; ++u) {
        float kf[DPL];
        kr[u].to_float(kf);
        float s = 0.f;
#pragma unroll
        for (int t = 0; t < DPL; ++t) s = fmaf(qf[t], kf[t], s);
        sc[u] = s;
      }
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
#pragma unroll
        for (int u = 0; u < kKeysPerGroup; ++u) sc[u] += __shfl_xor_sync(0xFFFFFFFFu, sc[u], o);
      }
      // one reference move per step: all keys of the step are added against the same maximum
      float mn = acc.m;
#pragma unroll
      for (int u = 0; u < kKeysPerGroup; ++u) mn = fmaxf(mn, valid[u] ? sc[u] : -CUDART_INF_F);
      if (mn != -CUDART_INF_F) {
        const float a = fast_ex2(acc.m - mn);                // m = -inf: 2^-inf = 0
        float pr[kKeysPerGroup], ps = 0.f;
#pragma unroll
        for (int u = 0; u < kKeysPerGroup; ++u) { pr[u] = valid[u] ? fast_ex2(sc[u] - mn) : 0.f; ps += pr[u]; }
        acc.l = acc.l * a + ps;
#pragma unroll
        for (int t = 0; t < DPL; ++t) acc.o[t] *= a;
#pragma unroll
        for (int u = 0; u < kKeysPerGroup; ++u) {
          float vf[DPL];
          vr[u].to_float(vf);
#pragma unroll
          for (int t = 0; t < DPL; ++t) acc.o[t] = fmaf(pr[u], vf[t], acc.o[t]);
        }
        acc.m = mn;
      }
    }
  }
  // ---- merge: the 4 lane groups of the warp, then the warps of the block
  acc.merge_xor(8);
  acc.merge_xor(16);
  if (g == 0) {
#pragma unroll
    for (int t = 0; t < DPL; ++t) sm_o[warp][sub * DPL + t] = acc.o[t];
    if (sub == 0) { sm_m[warp] = acc.m; sm_l[warp] = acc.l; }
  }
  __syncthreads();
  float mx = -CUDART_INF_F;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) mx = fmaxf(mx, sm_m[w]);
  float lt = 0.f;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) lt += sm_m[w] == -CUDART_INF_F ? 0.f : sm_l[w] * fast_ex2(sm_m[w] - mx);
  for (int t = tid; t < D; t += blockDim.x) {
    float ot = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) ot += sm_m[w] == -CUDART_INF_F ? 0.f : sm_o[w][t] * fast_ex2(sm_m[w] - mx);
    orow[t] = from_float<T>(lt > 0.f ? ot / lt : 0.f);
  }
  if (tid == 0) *lse_p = lt > 0.f ? (mx + log2f(lt)) * 0.6931471805599453f : -CUDART_INF_F;
}

}  // namespace

cudaError_t dam_launch_decode(const void* q, const void* K, const void* V, const void* blob, const dam_shape_t* s,
                              const int32_t* pos_dev, float scale, void* O, float* lse, void* scratch, cudaStream_t st) {
  // bf16 with a GQA group of at most 8 heads: one block per (sequence, KV head) on the tensor cores
  const cudaError_t ge = dam_launch_decode_group(q, K, V, blob, s, pos_dev, scale, O, lse, scratch, st);
  if (ge != cudaErrorNotSupported) return ge;
  const dim3 grid((unsigned)s->num_q_heads, (unsigned)s->num_seqs);
  const int group = s->num_q_heads / s->num_kv_heads;
  const float sl2 = scale * 1.4426950408889634f;
  uint32_t* status = reinterpret_cast<uint32_t*>(scratch) + 1;
  const unsigned char* bl = reinterpret_cast<const unsigned char*>(blob);
#define DAM_DECODE_LAUNCH(T, D)                                                                                  \
  decode_kernel<T, D><<<grid, kWarps * 32, 0, st>>>(reinterpret_cast<const T*>(q), reinterpret_cast<const T*>(K), \
                                                    reinterpret_cast<const T*>(V), bl, s->cu_seqlens_dev, pos_dev, \
                                                    s->num_seqs, s->num_q_heads, group, s->k_stride_tok,          \
                                                    s->k_stride_head, s->v_stride_tok, s->v_stride_head, sl2,     \
                                                    reinterpret_cast<T*>(O), lse, status)
  if (s->dtype == DAM_BF16 && s->head_dim == 128) DAM_DECODE_LAUNCH(__nv_bfloat16, 128);
  else if (s->dtype == DAM_BF16 && s->head_dim == 64) DAM_DECODE_LAUNCH(__nv_bfloat16, 64);
  else if (s->dtype == DAM_F32 && s->head_dim == 128) DAM_DECODE_LAUNCH(float, 128);
  else if (s->dtype == DAM_F32 && s->head_dim == 64) DAM_DECODE_LAUNCH(float, 64);
  else return cudaErrorNotSupported;
#undef DAM_DECODE_LAUNCH
  return cudaGetLastError();
}
