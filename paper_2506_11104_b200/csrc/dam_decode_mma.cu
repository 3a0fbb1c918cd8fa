// Generation-time attention under the stored patterns, bf16, for the query heads of one KV head at once
// (paper Sec. 4.3, Case 2, applied to one new token per sequence).
//
// The query heads of a GQA group read the same K / V rows, each under its own patterns.  One block takes one
// (sequence, KV head): it expands the pattern words of all the group's heads into ONE key list (the union, each key
// with a bit per head that says whether that head keeps it), brings the K and V rows of the list into shared memory
// with asynchronous copies (every row crosses from L2 once per group instead of once per head, and the bytes in
// flight are not bounded by registers), and computes with the warp-level tensor-core instruction: the group's
// queries are rows 0..G-1 of an m16 tile, so S = Q K^T of 16 keys costs 8 (head_dim 128) instructions for all heads
// together, and O += P V another 16, with no conversion of K or V to fp32 on the way.  A key that a head does not
// keep gets -inf before the softmax of that head's column (probability exactly 0).  Each warp walks its own chunks
// of 16 keys with a running softmax per head; the warps are merged through shared memory at the end.
//
// This is a gather of a few hundred 256-byte rows per head: bound by HBM / L2 bandwidth and latency, not by the
// tensor cores, which is why the small synchronous MMA shape serves (a 128-row tcgen05 tile would be 97 % padding).
#include <cuda_bf16.h>
#include <math_constants.h>

#include "dam_internal.cuh"

namespace {

constexpr int kGWarps = 5;            // warps per block
constexpr int kGStages = 1;           // chunks of 16 keys a warp holds in shared memory; with 1 a warp waits for its own copy and
                                      // the other 15 warps of the SM cover the wait (measured faster than 2 stages at half the occupancy)
constexpr int kGMinBlocks = 4;         // resident blocks per SM the register limit is sized for
constexpr int kGChunk = 16;           // keys per chunk (the K dimension of the P V instruction)
constexpr int kGRoundWords = 128;     // pattern words expanded per round (at most 4096 keys)
constexpr int kGMaxGroup = 8;         // query heads per KV head this kernel takes (rows 0..7 of the m16 tile)

__device__ __forceinline__ float g_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// K / V rows are read once per launch: they are marked to leave L2 first, so that the few lines every launch reads
// again (blob header, sequence records, pattern words, queries) are still there next time
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_evict_last_policy() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint32_t ldg_keep(const uint32_t* ptr, uint64_t policy) {
  uint32_t v;
  asm volatile("ld.global.nc.L2::cache_hint.u32 %0, [%1], %2;" : "=r"(v) : "l"(ptr), "l"(policy));
  return v;
}
// bits [x, x + 32) of a bit array of nwords words, zero outside it (x may be negative)
__device__ __forceinline__ uint32_t window32_keep(const uint32_t* bits, int nwords, int x, uint64_t policy) {
  const int w = x >> 5, sh = x & 31;
  const uint32_t lo = (w >= 0 && w < nwords) ? ldg_keep(bits + w, policy) : 0u;
  const uint32_t hi = (w + 1 >= 0 && w + 1 < nwords) ? ldg_keep(bits + w + 1, policy) : 0u;
  return __funnelshift_r(lo, hi, sh);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint64_t policy) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t* r) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16 x 8, fp32) += A (16 x 16, bf16, row-major) * B (16 x 8, bf16, column-major)
__device__ __forceinline__ void mma_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transpose of an 8 x 8 matrix of 16-bit elements held one row pair per lane (the accumulator layout of two columns)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

template <int D>
struct GLayout {
  static constexpr int row_bytes = D * 2;
  // rows are not padded: the 16-byte piece p of row r sits at piece p ^ (r & 7), so that the 8 rows of an ldmatrix
  // (same logical piece) fall into 8 different bank groups
  static constexpr int part_bytes = kGChunk * row_bytes;            // the K (or V) rows of one chunk
  static constexpr int stage_bytes = 2 * part_bytes;
  static constexpr int stages_total = kGWarps * kGStages * stage_bytes;
  static constexpr int merge_bytes = kGWarps * kGMaxGroup * (D + 2) * 4;   // per warp and head: O row, m, l
  static constexpr int work_bytes = stages_total > merge_bytes ? stages_total : merge_bytes;   // the merge reuses the stages
  static constexpr int codes_off = work_bytes;                              // u16 per listed key: round-local word * 32 + bit
  static constexpr int words_off = codes_off + kGRoundWords * 32 * 2;       // u32 [head][round-local word]: the round's pattern words
  static constexpr int total = words_off + kGMaxGroup * kGRoundWords * 4;
};

template <int D>
__global__ void __launch_bounds__(kGWarps * 32, kGMinBlocks)
decode_group_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ K,
                    const __nv_bfloat16* __restrict__ V, const unsigned char* __restrict__ blob,
                    const int32_t* __restrict__ cu, const int32_t* __restrict__ pos_dev, int num_seqs, int Hq, int G,
                    int64_t kst, int64_t ksh, int64_t vst, int64_t vsh, float scale_log2,
                    __nv_bfloat16* __restrict__ O, float* __restrict__ lse, uint32_t* status) {
  using LY = GLayout<D>;
  constexpr int KS = D / 16;                 // k-steps of S = Q K^T
  constexpr int kThreads = kGWarps * 32;
  extern __shared__ __align__(16) unsigned char gsm[];
  __shared__ int warp_tot[kGWarps];
  unsigned short* codes = reinterpret_cast<unsigned short*>(gsm + LY::codes_off);
  uint32_t* whs = reinterpret_cast<uint32_t*>(gsm + LY::words_off);
  const int kvh = blockIdx.x, b = blockIdx.y, h0 = kvh * G;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, row = lane >> 2, quad = lane & 3;
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  // the header, the position and the sequence bounds are requested together (one round trip to memory, not three)
  const int pos = __ldg(pos_dev + b), cu0 = __ldg(cu + b), cu1 = __ldg(cu + b + 1);
  const bool bad = H->magic != DAM_MAGIC || H->num_seqs != num_seqs || H->num_q_heads != Hq || pos < 0 || pos >= cu1 - cu0;
  if (bad) {
    if (tid == 0) atomicMax(status, (uint32_t)DAM_ERR_INVALID_ARGUMENT);
    for (int t = tid; t < G * D; t += kThreads) O[((int64_t)b * Hq + h0) * D + t] = __float2bfloat16_rn(0.f);
    if (tid < G) lse[(int64_t)b * Hq + h0 + tid] = -CUDART_INF_F;
    return;
  }
  const DamSeq sq = reinterpret_cast<const DamSeq*>(blob + H->off_seq)[b];
  const int L = sq.L, W = sq.W;
  const bool in_window = pos < L;
  // index space of pattern words: [0, W) the row of the true mask (inside the window) or the matched columns;
  // [W, 2W) the matched diagonals (below the window only)
  const int nwords = in_window ? W : 2 * W;
  const __nv_bfloat16* Kb = K + (int64_t)cu0 * kst + (int64_t)kvh * ksh;
  const __nv_bfloat16* Vb = V + (int64_t)cu0 * vst + (int64_t)kvh * vsh;

  // the group's queries as B fragments of Q^T (k = dimension, n = head h0 + n; columns G..7 are zero)
  uint32_t qa0[KS], qa2[KS];
  {
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((int64_t)b * Hq + h0 + (row < G ? row : 0)) * D);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa0[ks] = row < G ? __ldg(qrow + ks * 8 + quad) : 0u;
      qa2[ks] = row < G ? __ldg(qrow + ks * 8 + 4 + quad) : 0u;
    }
  }
  // this lane's heads are 2 * quad and 2 * quad + 1: running maximum (log2 domain) and the lane's share of the sum
  float m[2] = {-CUDART_INF_F, -CUDART_INF_F}, l[2] = {0.f, 0.f};
  float oacc[KS][4];                         // O^T: [t][0..1] = dimension 16 t + row, heads 2 quad + {0, 1}; [t][2..3] = dimension + 8
#pragma unroll
  for (int t = 0; t < KS; ++t) { oacc[t][0] = oacc[t][1] = oacc[t][2] = oacc[t][3] = 0.f; }

  const uint32_t stage0 = static_cast<uint32_t>(__cvta_generic_to_shared(gsm)) + warp * (kGStages * LY::stage_bytes);
  const uint64_t stream_policy = l2_evict_first_policy(), keep_policy = l2_evict_last_policy();
  for (int w0 = 0; w0 < nwords; w0 += kGRoundWords) {
    // ---- one key list for the whole group: a thread per pattern word, the words of all heads OR-ed.  A listed key
    //      is stored as (word, bit) of the round; which heads keep it is read back from the round's words
    const int wi = w0 + tid;                                // (threads beyond the round's words hold no word)
    uint32_t wh[kGMaxGroup], uni = 0u;
#pragma unroll
    for (int g = 0; g < kGMaxGroup; ++g) {
      wh[g] = 0u;
      if (g < G && tid < kGRoundWords && wi < nwords) {
        const DamHeadBits hb = dam_head_bits(blob, H, sq, h0 + g);
        if (in_window) {
          wh[g] = ldg_keep(hb.M + (size_t)pos * W + wi, keep_policy);
        } else if (wi < W) {
          wh[g] = ldg_keep(hb.V + wi, keep_policy);
        } else {
          // diagonal r = 32 (wi - W) + k selects key pos - r; dropped when that key is a matched column of the head
          // (then it is in the list already): bit k of the reversed 32-bit window of V that ends at key pos - 32 (wi - W)
          const int r0 = 32 * (wi - W);
          wh[g] = ldg_keep(hb.D + (wi - W), keep_policy) & ~__brev(window32_keep(hb.V, W, pos - r0 - 31, keep_policy));
        }
        uni |= wh[g];
      }
    }
    const int cnt = __popc(uni);
    int off = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xFFFFFFFFu, off, o);
      if (lane >= o) off += y;
    }
    __syncthreads();                                        // the previous round's list is no longer read
    if (lane == 31) warp_tot[warp] = off;
    if (tid < kGRoundWords) {
#pragma unroll
      for (int g = 0; g < kGMaxGroup; ++g) whs[g * kGRoundWords + tid] = wh[g];
    }
    __syncthreads();
    int total = 0, before = 0;
#pragma unroll
    for (int w = 0; w < kGWarps; ++w) {
      const int wt = warp_tot[w];
      if (w < warp) before += wt;
      total += wt;
    }
    off += before - cnt;
    while (uni) {
      const int k = __ffs(uni) - 1;
      uni &= uni - 1u;
      codes[off++] = (unsigned short)(tid * 32 + k);
    }
    __syncthreads();
    // key index of a listed key
    auto key_of = [&](uint32_t code) -> int {
      const int w = w0 + (int)(code >> 5), k = (int)(code & 31u);
      return (in_window || w < W) ? 32 * w + k : pos - (32 * (w - W) + k);
    };

    // ---- chunks of 16 keys, dealt to the warps round robin; a warp copies chunk i + 1 while it works on chunk i
    const int nchunks = (total + kGChunk - 1) / kGChunk;
    auto issue = [&](int c, int stage) {
      const uint32_t dstK = stage0 + stage * LY::stage_bytes, dstV = dstK + LY::part_bytes;
      constexpr int PPR = LY::row_bytes / 16;               // 16-byte pieces per row
#pragma unroll
      for (int i = 0; i < kGChunk * PPR / 32; ++i) {
        const int p = lane + 32 * i, r = p / PPR, piece = p % PPR;
        const int idx = c * kGChunk + r;
        const int j = key_of(codes[idx < total ? idx : c * kGChunk]);  // rows past the end repeat the chunk's first key (masked below)
        const uint32_t at = r * LY::row_bytes + ((piece ^ (r & 7)) << 4);
        cp_async16(dstK + at, Kb + (int64_t)j * kst + piece * 8, stream_policy);
        cp_async16(dstV + at, Vb + (int64_t)j * vst + piece * 8, stream_policy);
      }
    };
    // (a group is committed every time, also when there is no chunk left to copy, so that "all but the newest
    // kGStages - 1 groups are complete" always means "this iteration's chunk has landed")
#pragma unroll
    for (int pre = 0; pre < kGStages - 1; ++pre) {
      if (warp + pre * kGWarps < nchunks) issue(warp + pre * kGWarps, pre);
      cp_async_commit();
    }
    int it = 0;
    for (int c = warp; c < nchunks; c += kGWarps, ++it) {
      const int stage = it % kGStages;
      if (c + (kGStages - 1) * kGWarps < nchunks) issue(c + (kGStages - 1) * kGWarps, (it + kGStages - 1) % kGStages);
      cp_async_commit();
      cp_async_wait<kGStages - 1>();
      __syncwarp();
      const uint32_t sK = stage0 + stage * LY::stage_bytes, sV = sK + LY::part_bytes;
      // S^T = K Q^T for the 16 keys: this lane gets keys `row` and `row + 8` against its two heads
      float st[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t a4[4];
        ldmatrix_x4(sK + (((lane >> 3) & 1) * 8 + (lane & 7)) * LY::row_bytes + (((2 * ks + (lane >> 4)) ^ (lane & 7)) << 4), a4);
        mma_16816(st, a4, qa0[ks], qa2[ks]);
      }
      const int idx0 = c * kGChunk + row, idx1 = idx0 + 8;
      const uint32_t c0 = idx0 < total ? codes[idx0] : 0xFFFFu, c1 = idx1 < total ? codes[idx1] : 0xFFFFu;
      float alpha[2], p0[2], p1[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const uint32_t* wg = whs + (2 * quad + e) * kGRoundWords;         // the round's words of head 2 quad + e
        const bool k0 = c0 != 0xFFFFu && ((wg[c0 >> 5] >> (c0 & 31u)) & 1u);
        const bool k1 = c1 != 0xFFFFu && ((wg[c1 >> 5] >> (c1 & 31u)) & 1u);
        const float v0 = k0 ? st[e] * scale_log2 : -CUDART_INF_F;
        const float v1 = k1 ? st[2 + e] * scale_log2 : -CUDART_INF_F;
        float mx = fmaxf(v0, v1);
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 16));
        const float mn = fmaxf(m[e], mx);
        alpha[e] = 1.f; p0[e] = 0.f; p1[e] = 0.f;
        if (mn != -CUDART_INF_F) {
          alpha[e] = g_ex2(m[e] - mn);                       // m = -inf: 2^-inf = 0
          p0[e] = g_ex2(v0 - mn);
          p1[e] = g_ex2(v1 - mn);
          m[e] = mn;
        }
        l[e] = l[e] * alpha[e] + p0[e] + p1[e];
      }
      if (__any_sync(0xFFFFFFFFu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
        for (int t = 0; t < KS; ++t) { oacc[t][0] *= alpha[0]; oacc[t][1] *= alpha[1]; oacc[t][2] *= alpha[0]; oacc[t][3] *= alpha[1]; }
      }
      // P^T as B fragments (k = key, n = head): the transposes of the two 8 x 8 blocks [key][head] this warp holds
      __nv_bfloat162 pk0 = __floats2bfloat162_rn(p0[0], p0[1]), pk1 = __floats2bfloat162_rn(p1[0], p1[1]);
      const uint32_t pb0 = movmatrix_trans(*reinterpret_cast<uint32_t*>(&pk0));
      const uint32_t pb1 = movmatrix_trans(*reinterpret_cast<uint32_t*>(&pk1));
      // O^T += V^T P^T: V rows are [key][d]; the transposing load hands out A fragments (m = dimension, k = key)
#pragma unroll
      for (int t = 0; t < KS; ++t) {
        uint32_t a4[4];
        ldmatrix_x4_trans(sV + ((lane >> 4) * 8 + (lane & 7)) * LY::row_bytes + (((2 * t + ((lane >> 3) & 1)) ^ (lane & 7)) << 4), a4);
        mma_16816(oacc[t], a4, pb0, pb1);
      }
      __syncwarp();                                          // the stage is free for the copy the next iteration issues
    }
  }

  // ---- merge: the eight lanes with the same `quad` hold disjoint keys' sums of the same two heads; then the warps
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    l[e] += __shfl_xor_sync(0xFFFFFFFFu, l[e], 4);
    l[e] += __shfl_xor_sync(0xFFFFFFFFu, l[e], 8);
    l[e] += __shfl_xor_sync(0xFFFFFFFFu, l[e], 16);
  }
  __syncthreads();                                           // every warp is done with its stages: reuse them
  float* mg = reinterpret_cast<float*>(gsm);                 // [warp][head][D + 2]
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int g = 2 * quad + e;
    if (g < G) {
      float* dst = mg + ((size_t)warp * kGMaxGroup + g) * (D + 2);
#pragma unroll
      for (int t = 0; t < KS; ++t) { dst[16 * t + row] = oacc[t][e]; dst[16 * t + row + 8] = oacc[t][2 + e]; }
      if (row == 0) { dst[D] = m[e]; dst[D + 1] = l[e]; }
    }
  }
  __syncthreads();
  for (int e = tid; e < G * D; e += kThreads) {
    const int g = e / D, t = e % D;
    float mxw = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kGWarps; ++w) mxw = fmaxf(mxw, mg[((size_t)w * kGMaxGroup + g) * (D + 2) + D]);
    float lt = 0.f, ot = 0.f;
#pragma unroll
    for (int w = 0; w < kGWarps; ++w) {
      const float* src = mg + ((size_t)w * kGMaxGroup + g) * (D + 2);
      const float f = src[D] == -CUDART_INF_F ? 0.f : g_ex2(src[D] - mxw);
      lt += src[D + 1] * f;
      ot += src[t] * f;
    }
    O[((int64_t)b * Hq + h0 + g) * D + t] = __float2bfloat16_rn(lt > 0.f ? ot / lt : 0.f);
    if (t == 0) lse[(int64_t)b * Hq + h0 + g] = lt > 0.f ? (mxw + log2f(lt)) * 0.6931471805599453f : -CUDART_INF_F;
  }
}

}  // namespace

// bf16, head_dim 64 or 128, at most 8 query heads per KV head; cudaErrorNotSupported otherwise (the caller then
// takes the one-head-per-block kernel)
cudaError_t dam_launch_decode_group(const void* q, const void* K, const void* V, const void* blob, const dam_shape_t* s,
                                    const int32_t* pos_dev, float scale, void* O, float* lse, void* scratch,
                                    cudaStream_t st) {
  const int G = s->num_q_heads / s->num_kv_heads;
  if (s->dtype != DAM_BF16 || (s->head_dim != 64 && s->head_dim != 128) || G > kGMaxGroup) return cudaErrorNotSupported;
  int dev = 0;
  DamDeviceInfo di;
  cudaError_t e;
  if ((e = dam_current_device(&dev, &di)) != cudaSuccess) return e;
  const int smem = s->head_dim == 128 ? GLayout<128>::total : GLayout<64>::total;
  if (di.smem_optin < smem) return cudaErrorNotSupported;
  if ((e = dam_device_table().once(dev, DAM_SETUP_DECODE_SMEM, [](void) -> cudaError_t {
         cudaError_t r = cudaFuncSetAttribute(decode_group_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, GLayout<128>::total);
         if (r != cudaSuccess) return r;
         return cudaFuncSetAttribute(decode_group_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, GLayout<64>::total);
       })) != cudaSuccess)
    return e;
  const dim3 grid((unsigned)s->num_kv_heads, (unsigned)s->num_seqs);
  const float sl2 = scale * 1.4426950408889634f;
  uint32_t* status = reinterpret_cast<uint32_t*>(scratch) + 1;
  const __nv_bfloat16 *qq = reinterpret_cast<const __nv_bfloat16*>(q), *kk = reinterpret_cast<const __nv_bfloat16*>(K),
                      *vv = reinterpret_cast<const __nv_bfloat16*>(V);
  const unsigned char* bl = reinterpret_cast<const unsigned char*>(blob);
  if (s->head_dim == 128)
    decode_group_kernel<128><<<grid, kGWarps * 32, smem, st>>>(qq, kk, vv, bl, s->cu_seqlens_dev, pos_dev, s->num_seqs,
                                                               s->num_q_heads, G, s->k_stride_tok, s->k_stride_head,
                                                               s->v_stride_tok, s->v_stride_head, sl2,
                                                               reinterpret_cast<__nv_bfloat16*>(O), lse, status);
  else
    decode_group_kernel<64><<<grid, kGWarps * 32, smem, st>>>(qq, kk, vv, bl, s->cu_seqlens_dev, pos_dev, s->num_seqs,
                                                              s->num_q_heads, G, s->k_stride_tok, s->k_stride_head,
                                                              s->v_stride_tok, s->v_stride_head, sl2,
                                                              reinterpret_cast<__nv_bfloat16*>(O), lse, status);
  return cudaGetLastError();
}
