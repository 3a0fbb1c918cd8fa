// Stage-1 rule kernels: true-mask bits from a score tensor, diagonal / column counts, pattern
// match, tile classification and emission of the tile lists (paper Sec. 4.2.2 - 4.2.4, Sec. 4.3).
// Integer / bit work throughout; the only floating-point operations are the single compare
// p >= p* (equivalent to the Box-Cox threshold chain, see dam_api.cu) and one fp32 multiply +
// compare per pattern.
#include "dam_internal.cuh"

namespace {

// The rule kernels form a chain of short, dependent launches.  Each lets the next launch begin as soon as all
// of its own blocks are running (programmatic dependent launch) and then waits for the kernel before it to
// have completed with its memory visible: the launch latency of every link is hidden under its predecessor.
// Both instructions do nothing in a kernel that was launched the ordinary way.
__device__ __forceinline__ void dam_chain_prologue() {
  asm volatile("griddepcontrol.launch_dependents;");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = 0; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ const DamSeq* blob_seqs(const unsigned char* blob, const DamHeader* h) {
  return reinterpret_cast<const DamSeq*>(blob + h->off_seq);
}

// ---------------------------------------------------------------------------------------------
// Header + per-sequence table + q-block table, computed on the device from cu_seqlens so that no
// host buffer has to outlive the call.  One block.
// ---------------------------------------------------------------------------------------------
__global__ void init_blob_kernel(unsigned char* blob, DamHeader hdr, const int32_t* __restrict__ cu,
                                 int pcl_max, int Hq, int all_ones_causal /* -1: DAM mask */) {
  asm volatile("griddepcontrol.launch_dependents;");     // a kernel chained behind this one may start its prologue
  DamHeader* H = reinterpret_cast<DamHeader*>(blob);
  DamSeq* seqs = reinterpret_cast<DamSeq*>(blob + hdr.off_seq);
  int32_t* qbseq = reinterpret_cast<int32_t*>(blob + hdr.off_qbseq);
  uint32_t* pairtab = reinterpret_cast<uint32_t*>(blob + hdr.off_pairtab);
  if (threadIdx.x == 0) {
    *H = hdr;
    uint64_t dv = 0, tr = 0, po = 0, co = 0, go = 0, tb = 0;
    int fq = 0, fp = 0;
    const int gather = (hdr.flags & DAM_FLAG_GATHER) ? 1 : 0;
    for (int b = 0; b < hdr.num_seqs; ++b) {
      int t0 = cu[b], S = cu[b + 1] - t0;
      int L = S < pcl_max ? S : pcl_max;
      if (L < 0) L = 0;
      int W = L > 0 ? dam_words(L) : 0;
      int nL = (L + DAM_TILE - 1) / DAM_TILE;
      int nq = (S + DAM_TILE - 1) / DAM_TILE;
      DamSeq s;
      s.tok_start = t0; s.S = S; s.L = L; s.nq = nq;
      s.first_qblock = fq; s.W = W; s.nL = nL; s.first_pair = fp;
      s.dv_off = dv; s.true_off = tr; s.p_off = po; s.cnt_off = co; s.gath_off = go; s.tile_base = tb;
      seqs[b] = s;
      dv += (uint64_t)Hq * 3 * W;
      tr += (uint64_t)Hq * L * W;
      po += (uint64_t)Hq * L * L;
      if (all_ones_causal < 0) co += (uint64_t)Hq * dam_cnt_stride(L, W, nL);
      else co += all_ones_causal ? (uint64_t)nq * (nq + 1) / 2 : (uint64_t)nq * nq;   // tile base per head
      go += (uint64_t)Hq * nL;
      if (all_ones_causal < 0) tb += dam_row_tile_prefix(nq, nL, L, gather);
      fq += nq;
      fp += (nq + 1) / 2;
    }
    H->head_tile_cap = tb;
    if (all_ones_causal < 0) {
      // the tile lists have a fixed place per row (see the layout notes): nothing to compact, no sizes to wait for
      H->bytes_used = hdr.off_tiles + 4ull * Hq * tb;
      reinterpret_cast<uint32_t*>(blob + hdr.off_tile_ptr)[hdr.rows] = (uint32_t)(Hq * tb);
    }
  }
  __syncthreads();
  for (int b = 0; b < hdr.num_seqs; ++b) {
    int fq = seqs[b].first_qblock, nq = seqs[b].nq, fp = seqs[b].first_pair;
    for (int q = threadIdx.x; q < nq; q += blockDim.x) qbseq[fq + q] = b;
    for (int p = threadIdx.x; p < (nq + 1) / 2; p += blockDim.x)
      pairtab[fp + p] = (uint32_t)(fq + 2 * p) | ((2 * p + 1 < nq) ? 0x80000000u : 0u);
  }
}

// ---------------------------------------------------------------------------------------------
// True-mask bits from an fp32 map P ([L][L] per (seq, head)): bit = [P >= p*], forced to 0 above
// the diagonal.  One warp per (row, 32-column word); coalesced reads, one word written per warp.
// ---------------------------------------------------------------------------------------------
__global__ void bits_from_scores_kernel(unsigned char* blob, const float* __restrict__ P, float pstar) {
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int sh = blockIdx.y;
  const int b = sh / H->num_q_heads, h = sh % H->num_q_heads;
  const DamSeq sq = blob_seqs(blob, H)[b];
  if (sq.L == 0) return;
  uint32_t* M = reinterpret_cast<uint32_t*>(blob + H->off_true) + sq.true_off + (uint64_t)h * sq.L * sq.W;
  const float* Ph = P + sq.p_off + (uint64_t)h * sq.L * sq.L;
  const int lane = threadIdx.x & 31;
  const long long nitems = (long long)sq.L * sq.W;
  const long long wstride = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long it = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); it < nitems; it += wstride) {
    int i = (int)(it / sq.W), w = (int)(it % sq.W);
    int j = w * 32 + lane;
    float p = (j < sq.L && j <= i) ? __ldg(Ph + (size_t)i * sq.L + j) : 0.0f;
    uint32_t word = __ballot_sync(0xFFFFFFFFu, p >= pstar);
    if (lane == 0) M[(size_t)i * sq.W + w] = word;
  }
}

// Transpose of a 32 x 32 bit matrix held one row per lane: lane c returns column c (bit r = bit c of row r).
__device__ __forceinline__ uint32_t dam_transpose32(uint32_t x, int lane) {
#pragma unroll
  for (int j = 16; j >= 1; j >>= 1) {
    const uint32_t m = j == 16 ? 0x0000FFFFu : j == 8 ? 0x00FF00FFu : j == 4 ? 0x0F0F0F0Fu : j == 2 ? 0x33333333u : 0x55555555u;
    const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, j);
    x = (lane & j) ? ((x & ~m) | ((y >> j) & m)) : ((x & m) | ((y & m) << j));
  }
  return x;
}

// ---------------------------------------------------------------------------------------------
// Counts: one block per 128 x 128 tile (qb, kb <= qb) of the window.  Thread t owns row qb*128+t
// and its 128 bits.  Column counts (128), diagonal counts (255) and the tile's popcount are made per warp
// with bit-matrix transposes, summed in shared memory and flushed with integer atomics (order-independent).
// ---------------------------------------------------------------------------------------------
__global__ void counts_kernel(const unsigned char* blob, unsigned char* scratch, uint64_t off_cnt) {
  dam_chain_prologue();
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int sh = blockIdx.y;
  const int b = sh / H->num_q_heads, h = sh % H->num_q_heads;
  const DamSeq sq = blob_seqs(blob, H)[b];
  const int nL = sq.nL;
  // tile index -> (qb, kb) over the lower triangle
  int t = blockIdx.x;
  if (t >= nL * (nL + 1) / 2) return;
  int qb = (int)((sqrtf(8.0f * t + 1.0f) - 1.0f) * 0.5f);
  while ((qb + 1) * (qb + 2) / 2 <= t) ++qb;
  while (qb * (qb + 1) / 2 > t) --qb;
  const int kb = t - qb * (qb + 1) / 2;

  const uint32_t* M = reinterpret_cast<const uint32_t*>(blob + H->off_true) + sq.true_off + (uint64_t)h * sq.L * sq.W;
  int32_t* cnt = reinterpret_cast<int32_t*>(scratch + off_cnt) + sq.cnt_off + (uint64_t)h * dam_cnt_stride(sq.L, sq.W, nL);
  int32_t* cntD = cnt;
  int32_t* cntV = cnt + sq.L;
  int32_t* tile_pop = cnt + 2 * sq.L + 2 * (sq.W + 1);

  __shared__ int sV[DAM_TILE];
  __shared__ int sD[2 * DAM_TILE];
  __shared__ int sPop;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int i = qb * DAM_TILE + tid;
  uint4 bits = make_uint4(0, 0, 0, 0);
  if (i < sq.L) bits = __ldg(reinterpret_cast<const uint4*>(M + (size_t)i * sq.W + kb * 4));
  const int nz = (bits.x | bits.y | bits.z | bits.w) != 0;
  if (!__syncthreads_or(nz)) return;
  sV[tid] = 0; sD[tid] = 0; sD[tid + DAM_TILE] = 0;
  if (tid == 0) sPop = 0;
  __syncthreads();
  // The patterns being counted are whole columns and whole diagonals, i.e. the same counter for every row: a
  // counter update per set bit would serialise.  Instead every warp transposes its 32 x 32 bit blocks with
  // shuffles, so that lane c holds column c of the block and one population count gives the column's count.
  // Diagonals are columns of the rows reversed and shifted by the row index: bit 127 + row - c of a 160-bit row.
  if (__any_sync(0xFFFFFFFFu, nz)) {
    const uint32_t w[4] = {bits.x, bits.y, bits.z, bits.w};
    int pop = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      pop += __popc(w[q]);
      if (__any_sync(0xFFFFFFFFu, w[q] != 0u)) {
        const int n = __popc(dam_transpose32(w[q], lane));
        if (n) atomicAdd(&sV[q * 32 + lane], n);
      }
    }
    const uint32_t rev[4] = {__brev(w[3]), __brev(w[2]), __brev(w[1]), __brev(w[0])};   // bit 127 - c
    uint32_t R[5];
    R[0] = rev[0] << lane;
#pragma unroll
    for (int k = 1; k < 4; ++k) R[k] = __funnelshift_l(rev[k - 1], rev[k], lane);
    R[4] = __funnelshift_l(rev[3], 0u, lane);
#pragma unroll
    for (int k = 0; k < 5; ++k) {
      if (__any_sync(0xFFFFFFFFu, R[k] != 0u)) {
        const int n = __popc(dam_transpose32(R[k], lane));
        if (n) atomicAdd(&sD[warp * 32 + k * 32 + lane], n);       // index row_in_tile - c + 127
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) pop += __shfl_xor_sync(0xFFFFFFFFu, pop, o);
    if (lane == 0) atomicAdd(&sPop, pop);
  }
  __syncthreads();
  {
    int c = kb * DAM_TILE + tid;
    if (sV[tid] && c < sq.L) atomicAdd(&cntV[c], sV[tid]);
    for (int idx = tid; idx < 2 * DAM_TILE - 1; idx += DAM_TILE) {
      int r = (qb - kb) * DAM_TILE + idx - (DAM_TILE - 1);
      if (sD[idx] && r >= 0 && r < sq.L) atomicAdd(&cntD[r], sD[idx]);
    }
    if (tid == 0) tile_pop[qb * nL + kb] = sPop;
  }
}

// ---------------------------------------------------------------------------------------------
// Match: D[r] = [cntD[r] >= mu * (L - r)], V[c] likewise (one fp32 multiply, one compare), written
// as bit sets; Drev = D reversed; prefix popcounts per word for range queries.  Block per (seq, head).
// ---------------------------------------------------------------------------------------------
__global__ void match_kernel(unsigned char* blob, unsigned char* scratch, uint64_t off_cnt, float mu, int min_support) {
  dam_chain_prologue();
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int sh = blockIdx.x;
  const int b = sh / H->num_q_heads, h = sh % H->num_q_heads;
  const DamSeq sq = blob_seqs(blob, H)[b];
  if (sq.L == 0) return;
  const int L = sq.L, W = sq.W;
  uint32_t* dv = reinterpret_cast<uint32_t*>(blob + H->off_dv) + sq.dv_off + (uint64_t)h * 3 * W;
  uint32_t* Dw = dv; uint32_t* Rw = dv + W; uint32_t* Vw = dv + 2 * W;
  int32_t* cnt = reinterpret_cast<int32_t*>(scratch + off_cnt) + sq.cnt_off + (uint64_t)h * dam_cnt_stride(L, W, sq.nL);
  const int32_t* cntD = cnt;
  const int32_t* cntV = cnt + L;
  int32_t* prefD = cnt + 2 * L;
  int32_t* prefV = prefD + (W + 1);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int w = warp; w < W; w += nw) {
    int k = w * 32 + lane;
    bool d = false, v = false;
    if (k < L) {
      int size = L - k;
      float need = __fmul_rn(mu, (float)size);
      bool ok = size >= min_support;
      d = ok && ((float)cntD[k] >= need);
      v = ok && ((float)cntV[k] >= need);
    }
    uint32_t dw = __ballot_sync(0xFFFFFFFFu, d), vw = __ballot_sync(0xFFFFFFFFu, v);
    if (lane == 0) { Dw[w] = dw; Vw[w] = vw; }
  }
  __threadfence_block();
  __syncthreads();
  for (int w = warp; w < W; w += nw) {
    int x = w * 32 + lane;
    int src = L - 1 - x;
    bool bit = (x < L) && ((Dw[src >> 5] >> (src & 31)) & 1u);
    uint32_t rw = __ballot_sync(0xFFFFFFFFu, bit);
    if (lane == 0) Rw[w] = rw;
  }
  if (warp == 0) {
    // prefix popcounts per word (exclusive), 32 words at a time
    int runD = 0, runV = 0;
    for (int w0 = 0; w0 < W; w0 += 32) {
      const int w = w0 + lane;
      int pd = w < W ? __popc(Dw[w]) : 0, pv = w < W ? __popc(Vw[w]) : 0;
      int id = pd, iv = pv;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int yd = __shfl_up_sync(0xFFFFFFFFu, id, o), yv = __shfl_up_sync(0xFFFFFFFFu, iv, o);
        if (lane >= o) { id += yd; iv += yv; }
      }
      if (w < W) { prefD[w] = runD + id - pd; prefV[w] = runV + iv - pv; }
      runD += __shfl_sync(0xFFFFFFFFu, id, 31);
      runV += __shfl_sync(0xFFFFFFFFu, iv, 31);
    }
    if (lane == 0) { prefD[W] = runD; prefV[W] = runV; }
  }
}

// ---------------------------------------------------------------------------------------------
// Tile classification.  One warp per row = (head, global q-block); lanes test candidate kv tiles in
// ascending order and writes the kept ones into the pair's fixed range of tiles[] (one pass: nothing is counted
// first, nothing is compacted afterwards).
// ---------------------------------------------------------------------------------------------
struct HeadView {
  const uint32_t* Dw; const uint32_t* Vw;
  const int32_t* prefD; const int32_t* prefV; const int32_t* tile_pop;
  int L, W, nL, S;
};

__device__ __forceinline__ int cnt_below(const uint32_t* bits, const int32_t* pref, int x) {
  int w = x >> 5, s = x & 31;
  int c = pref[w];
  if (s) c += __popc(bits[w] & ((1u << s) - 1u));
  return c;
}
__device__ __forceinline__ int cnt_range(const uint32_t* bits, const int32_t* pref, int lo, int hi) {
  return cnt_below(bits, pref, hi + 1) - cnt_below(bits, pref, lo);
}

// returns 0 (empty), DAM_KIND_FULL or DAM_KIND_PARTIAL
__device__ __forceinline__ uint32_t classify_tile(const HeadView& v, int qb, int kb) {
  const int i0 = qb * DAM_TILE;
  const int i1 = min(i0 + DAM_TILE, v.S);
  const int j0 = kb * DAM_TILE;
  bool act = false, full = false;
  if (i0 < v.L && j0 < v.L) {                       // rows inside the window: the true mask
    int pop = v.tile_pop[qb * v.nL + kb];
    act = pop > 0;
    full = pop == DAM_TILE * DAM_TILE;
  }
  if (i1 > v.L && v.L > 0) {                        // rows below the window: matched patterns
    const int a = max(i0, v.L);
    const bool whole = (a == i0) && (i1 - i0 == DAM_TILE) && (kb < qb);
    if (j0 < v.L) {
      int hi = min(j0 + DAM_TILE - 1, v.L - 1);
      int n = cnt_range(v.Vw, v.prefV, j0, hi);
      act |= n > 0;
      full |= whole && n == DAM_TILE;
    }
    int rlo = a - (j0 + DAM_TILE - 1), rhi = (i1 - 1) - j0;
    int clo = max(rlo, 0), chi = min(rhi, v.L - 1);
    if (clo <= chi) {
      int n = cnt_range(v.Dw, v.prefD, clo, chi);
      act |= n > 0;
      full |= whole && clo == rlo && chi == rhi && n == 2 * DAM_TILE - 1;
    }
  }
  return act ? (full ? DAM_KIND_FULL : DAM_KIND_PARTIAL) : 0u;
}

// Rows from 2L - 1 on with gathered columns: only the matched diagonals count (their keys are all >= L - 1
// while every matched column is < L and served by the gathered tiles).
__device__ __forceinline__ uint32_t classify_band(const HeadView& v, int qb, int kb) {
  const int i0 = qb * DAM_TILE;
  const int i1 = min(i0 + DAM_TILE, v.S);
  const int j0 = kb * DAM_TILE;
  const int rlo = i0 - (j0 + DAM_TILE - 1), rhi = (i1 - 1) - j0;
  const int clo = max(rlo, 0), chi = min(rhi, v.L - 1);
  if (clo > chi) return 0u;
  const int n = cnt_range(v.Dw, v.prefD, clo, chi);
  if (n == 0) return 0u;
  const bool whole = (i1 - i0 == DAM_TILE) && (kb < qb) && clo == rlo && chi == rhi;
  return (whole && n == 2 * DAM_TILE - 1) ? DAM_KIND_FULL : DAM_KIND_PARTIAL;
}

__global__ void classify_kernel(unsigned char* blob, unsigned char* scratch, uint64_t off_cnt, uint64_t off_items,
                                uint64_t off_keys) {
  dam_chain_prologue();
  DamHeader* H = reinterpret_cast<DamHeader*>(blob);
  const int lane = threadIdx.x & 31;
  const int prow = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // one warp per (head, q-block pair)
  // block totals of the three statistics: one global atomic per block instead of one per warp on the same address
  __shared__ unsigned long long s_mask_tiles;
  __shared__ uint32_t s_total, s_full;
  if (threadIdx.x == 0) { s_mask_tiles = 0ull; s_total = 0u; s_full = 0u; }
  __syncthreads();
  if (prow < H->prows) {
  const int h = prow / H->total_pairs, gp = prow % H->total_pairs;
  const uint32_t pt = reinterpret_cast<const uint32_t*>(blob + H->off_pairtab)[gp];
  const int gqb0 = (int)(pt & 0x7FFFFFFFu), nblk = (pt >> 31) ? 2 : 1;
  const int b = reinterpret_cast<const int32_t*>(blob + H->off_qbseq)[gqb0];
  const DamSeq sq = blob_seqs(blob, H)[b];
  HeadView v;
  const uint32_t* dv = reinterpret_cast<const uint32_t*>(blob + H->off_dv) + sq.dv_off + (uint64_t)h * 3 * sq.W;
  const int32_t* cnt = reinterpret_cast<const int32_t*>(scratch + off_cnt) + sq.cnt_off +
                       (uint64_t)h * dam_cnt_stride(sq.L, sq.W, sq.nL);
  v.Dw = dv; v.Vw = dv + 2 * sq.W;
  v.prefD = cnt + 2 * sq.L; v.prefV = v.prefD + (sq.W + 1); v.tile_pop = v.prefV + (sq.W + 1);
  v.L = sq.L; v.W = sq.W; v.nL = sq.nL; v.S = sq.S;
  uint32_t* tile_ptr = reinterpret_cast<uint32_t*>(blob + H->off_tile_ptr);
  uint32_t* tiles = reinterpret_cast<uint32_t*>(blob + H->off_tiles);
  const int gflag = (H->flags & DAM_FLAG_GATHER) ? 1 : 0;
  const int qb0 = gqb0 - sq.first_qblock;
  // the pair's fixed range of tiles[]: entries of block qb0, then of block qb0 + 1, then zeros
  const uint64_t head_base = (uint64_t)h * H->head_tile_cap + sq.tile_base;
  const uint32_t pair_begin = (uint32_t)(head_base + dam_row_tile_prefix(qb0, sq.nL, sq.L, gflag));
  const uint32_t pair_end = (uint32_t)(head_base + dam_row_tile_prefix(qb0 + nblk, sq.nL, sq.L, gflag));
  uint32_t base = pair_begin, a1 = pair_begin;
  int pair_total = 0, nfull = 0, mask_tiles = 0;
  // Per query block: candidates, ascending: [0, min(qb, nL-1)] then [max(that + 1, qb - nL), qb].  From row 2L - 1
  // on (gathered columns enabled) the first range is replaced by the gathered tiles and the second range is
  // classified on the matched diagonals alone.  The tiles of the mask itself (128 x 128 grid) with an active cell
  // are counted in the same sweep: they equal the listed tiles unless the row is served by gathered tiles.
  struct BlockPlan { int qb, gathered, n1, lo2, ncand, m1, l2, nmask; };
  const int nV = (gflag && sq.L > 0) ? v.prefV[sq.W] : 0;        // matched columns of the head
  BlockPlan plan[2];
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    BlockPlan& p = plan[x];
    p.qb = qb0 + x;
    p.gathered = gflag && sq.L > 0 && p.qb >= dam_gather_first_qblock(sq.L);
    p.n1 = p.gathered ? (nV + DAM_TILE - 1) / DAM_TILE : min(p.qb, sq.nL - 1) + 1;
    p.lo2 = p.gathered ? max(0, p.qb - sq.nL) : max(p.n1, p.qb - sq.nL);
    p.ncand = x < nblk ? p.n1 + max(0, p.qb - p.lo2 + 1) : 0;
    p.m1 = min(p.qb, sq.nL - 1) + 1;
    p.l2 = max(p.m1, p.qb - sq.nL);
    p.nmask = (x < nblk && p.gathered) ? p.m1 + max(0, p.qb - p.l2 + 1) : 0;
  }
  // one candidate per lane: list entry (kind 0: not listed) and whether the mask tile has an active cell
  auto eval = [&](const BlockPlan& p, int idx, uint32_t& kind, uint32_t& entry, bool& act) {
    kind = 0u; entry = 0u;
    if (idx < p.ncand) {
      if (p.gathered && idx < p.n1) {
        kind = DAM_KIND_GATHERED;
        entry = (uint32_t)idx | ((uint32_t)(min(DAM_TILE, nV - idx * DAM_TILE) - 1) << 16) | (kind << 28);
      } else {
        const int kb = idx < p.n1 ? idx : p.lo2 + (idx - p.n1);
        kind = p.gathered ? classify_band(v, p.qb, kb) : classify_tile(v, p.qb, kb);
        entry = (uint32_t)kb | (kind << 28);
      }
    }
    act = idx < p.nmask && classify_tile(v, p.qb, idx < p.m1 ? idx : p.l2 + (idx - p.m1)) != 0u;
  };
  int total = 0, nat = 0;
  auto consume = [&](uint32_t kind, uint32_t entry, bool act) {
    const uint32_t m = __ballot_sync(0xFFFFFFFFu, kind != 0);
    if (kind) {
      const int rank = __popc(m & ((1u << lane) - 1u));
      if (base + total + rank < pair_end) tiles[base + total + rank] = entry;     // always true: the range is the bound
    }
    nfull += __popc(__ballot_sync(0xFFFFFFFFu, kind == DAM_KIND_FULL || (kind == DAM_KIND_GATHERED && ((entry >> 16) & 0xFFu) == DAM_TILE - 1)));
    total += __popc(m);
    nat += __popc(__ballot_sync(0xFFFFFFFFu, act));
  };
  auto finish_block = [&](int x) {
    if (lane == 0) tile_ptr[h * H->total_qblocks + gqb0 + x] = base;
    base += total;
    if (x == 0) a1 = base;
    pair_total += total;
    mask_tiles += plan[x].gathered ? nat : total;
    total = 0; nat = 0;
  };
  const int span0 = max(plan[0].ncand, plan[0].nmask), span1 = max(plan[1].ncand, plan[1].nmask);
  if (span0 <= 64 && span1 <= 64) {
    // the usual sizes: all candidates of both blocks are looked up before any is written, so that their loads
    // (prefix counts, bit words, tile counts) are in flight together
    uint32_t k[4], e[4];
    bool a[4];
    eval(plan[0], lane, k[0], e[0], a[0]);
    eval(plan[0], 32 + lane, k[1], e[1], a[1]);
    eval(plan[1], lane, k[2], e[2], a[2]);
    eval(plan[1], 32 + lane, k[3], e[3], a[3]);
    consume(k[0], e[0], a[0]);
    if (span0 > 32) consume(k[1], e[1], a[1]);
    finish_block(0);
    if (nblk == 2) {
      consume(k[2], e[2], a[2]);
      if (span1 > 32) consume(k[3], e[3], a[3]);
      finish_block(1);
    }
  } else {
    for (int x = 0; x < nblk; ++x) {
      for (int c0 = 0; c0 < max(plan[x].ncand, plan[x].nmask); c0 += 32) {
        uint32_t kind, entry;
        bool act;
        eval(plan[x], c0 + lane, kind, entry, act);
        consume(kind, entry, act);
      }
      finish_block(x);
    }
  }
  // zero entries up to the next pair
  for (uint32_t t = base + lane; t < pair_end; t += 32) tiles[t] = 0u;
  if (lane == 0) {
    // the work item and its key (listed tiles): the ordering kernel moves the item to its place in the work list
    DamItem it;
    it.head = h; it.tok0 = sq.tok_start; it.qb0 = qb0; it.S = sq.S;
    it.a0 = pair_begin; it.a1 = a1; it.b1 = base;
    it.seq_hasB = (uint32_t)b | (nblk == 2 ? 0x80000000u : 0u);
    // index (pair, head): the order the pairs keep inside a bucket of the work list
    const size_t at = (size_t)gp * H->num_q_heads + h;
    reinterpret_cast<DamItem*>(scratch + off_items)[at] = it;
    reinterpret_cast<uint32_t*>(scratch + off_keys)[at] = (uint32_t)min(pair_total, DAM_HIST - 1);
    atomicAdd(&s_mask_tiles, (unsigned long long)mask_tiles);
    atomicAdd(&s_total, (uint32_t)pair_total);
    atomicAdd(&s_full, (uint32_t)nfull);
  }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (s_mask_tiles) atomicAdd(reinterpret_cast<unsigned long long*>(&H->mask_tiles), s_mask_tiles);
    if (s_total) atomicAdd(&H->total_tiles, s_total);
    if (s_full) atomicAdd(&H->full_tiles, s_full);
  }
}

// ---------------------------------------------------------------------------------------------
// Work order: the pairs are sorted by listed tiles, most first (a counting sort: histogram, exclusive scan,
// placement).  Blocks of 1024 threads; every block places 1024 pairs.
// ---------------------------------------------------------------------------------------------
__device__ uint32_t block_excl_scan(uint32_t x, uint32_t* total, uint32_t* sm /* 32 */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) sm[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t s = lane < (int)(blockDim.x >> 5) ? sm[lane] : 0u;      // blocks of fewer than 32 warps
    uint32_t si = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t y = __shfl_up_sync(0xFFFFFFFFu, si, o);
      if (lane >= o) si += y;
    }
    sm[lane] = si - s;
    if (lane == 31) *total = si;
  }
  __syncthreads();
  uint32_t r = sm[warp] + inc - x;
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(1024)
order_kernel(unsigned char* blob, unsigned char* scratch, uint64_t off_items, uint64_t off_keys) {
  dam_chain_prologue();
  DamHeader* H = reinterpret_cast<DamHeader*>(blob);
  __shared__ uint32_t sm[32];
  __shared__ uint32_t tot;
  __shared__ uint32_t start[DAM_HIST];      // pairs per key, then the first place of the key's bucket
  __shared__ uint32_t before[DAM_HIST];     // pairs per key that precede this block's share, then the running cursor
  const uint4* src = reinterpret_cast<const uint4*>(scratch + off_items);      // items in (pair, head) order
  const uint32_t* keys = reinterpret_cast<const uint32_t*>(scratch + off_keys);
  uint4* dst = reinterpret_cast<uint4*>(blob + H->off_work);
  const int prows = H->prows;
  for (int k = threadIdx.x; k < DAM_HIST; k += blockDim.x) { start[k] = 0u; before[k] = 0u; }
  __syncthreads();
  // Every block places blockDim.x pairs and needs nothing from the other blocks: it counts all pairs per key
  // itself, and those that precede its share.  Inside a bucket the pairs keep the order (pair, head): the query
  // heads of one KV head at the same pair of query blocks list the same kv tiles, and neighbours in the work
  // list run at the same time on different SMs, so the second to fourth find the K and V tiles in L2.  An item
  // is two 16-byte words: head, tok0, qb0, S | a0, a1, b1, seq_hasB; its key is the number of listed tiles.
  const int my_begin = blockIdx.x * (int)blockDim.x;
  // (in this order the lanes of a warp are the heads of one pair: their keys mostly differ, so plain shared-memory
  // atomics do not collide inside an instruction)
  auto count = [&](uint32_t* hist, uint32_t key) {
    if (key != 0xFFFFFFFFu) atomicAdd(&hist[key], 1u);
  };
  for (int i0 = 0; i0 < prows; i0 += 4 * (int)blockDim.x) {
    uint32_t k[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int idx = i0 + j * (int)blockDim.x + (int)threadIdx.x;
      k[j] = idx < prows ? keys[idx] : 0xFFFFFFFFu;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int idx0 = i0 + j * (int)blockDim.x;                  // first index of this warp-uniform batch
      count(start, k[j]);
      if (idx0 + (int)blockDim.x <= my_begin) count(before, k[j]);   // batches are aligned to the blocks' shares
    }
  }
  __syncthreads();
  // first place of every bucket: after all buckets with more tiles (descending order of the key)
  {
    const int per = (DAM_HIST + blockDim.x - 1) / blockDim.x;
    const int q0 = threadIdx.x * per, q1 = min(DAM_HIST, q0 + per);     // positions in descending-key order
    uint32_t local = 0;
    for (int k = q0; k < q1; ++k) local += start[DAM_HIST - 1 - k];
    uint32_t e = block_excl_scan(local, &tot, sm);
    for (int k = q0; k < q1; ++k) { const uint32_t c = start[DAM_HIST - 1 - k]; start[DAM_HIST - 1 - k] = e; e += c; }
  }
  __syncthreads();
  {
    const int idx = my_begin + (int)threadIdx.x;
    uint4 u = make_uint4(0u, 0u, 0u, 0u), v = u;
    uint32_t key = 0xFFFFFFFFu;
    if (idx < prows) { u = src[2 * (size_t)idx]; v = src[2 * (size_t)idx + 1]; key = keys[idx]; }
    if (key != 0xFFFFFFFFu) {
      const uint32_t pos = start[key] + atomicAdd(&before[key], 1u);
      dst[2 * (size_t)pos] = u; dst[2 * (size_t)pos + 1] = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// All-ones blob: every (causal: lower-triangular) tile listed as FULL.
// ---------------------------------------------------------------------------------------------
__global__ void all_ones_kernel(unsigned char* blob, int causal) {
  DamHeader* H = reinterpret_cast<DamHeader*>(blob);
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= H->rows) return;
  const int h = row / H->total_qblocks, gqb = row % H->total_qblocks;
  const int b = reinterpret_cast<const int32_t*>(blob + H->off_qbseq)[gqb];
  const DamSeq* seqs = blob_seqs(blob, H);
  const DamSeq sq = seqs[b];
  const DamSeq last = seqs[H->num_seqs - 1];
  const uint64_t per_head = last.cnt_off + (causal ? (uint64_t)last.nq * (last.nq + 1) / 2 : (uint64_t)last.nq * last.nq);
  const int qb = gqb - sq.first_qblock;
  const int n = causal ? qb + 1 : sq.nq;
  const uint64_t base = (uint64_t)h * per_head + sq.cnt_off + (causal ? (uint64_t)qb * (qb + 1) / 2 : (uint64_t)qb * sq.nq);
  uint32_t* tile_ptr = reinterpret_cast<uint32_t*>(blob + H->off_tile_ptr);
  uint32_t* tiles = reinterpret_cast<uint32_t*>(blob + H->off_tiles);
  for (int k = lane; k < n; k += 32) tiles[base + k] = (uint32_t)k | (DAM_KIND_FULL << 28);
  if (lane == 0) {
    tile_ptr[row] = (uint32_t)base;
    // pair order: heaviest q-blocks first (exact longest-first for one sequence)
    if (((qb & 1) == 0)) {
      const int gp = sq.first_pair + (qb >> 1);
      const bool hasB = qb + 1 < sq.nq;
      DamItem it;
      it.head = h; it.tok0 = sq.tok_start; it.qb0 = qb; it.S = sq.S;
      it.a0 = (uint32_t)base; it.a1 = it.a0 + n;
      it.b1 = it.a1 + (hasB ? (causal ? qb + 2 : sq.nq) : 0);
      it.seq_hasB = (uint32_t)b | (hasB ? 0x80000000u : 0u);
      reinterpret_cast<DamItem*>(blob + H->off_work)[(uint64_t)h * H->total_pairs + (H->total_pairs - 1 - gp)] = it;
    }
    if (row == H->rows - 1) {
      uint32_t tot = (uint32_t)(base + n);
      tile_ptr[H->rows] = tot;
      H->total_tiles = tot;
      H->full_tiles = tot;
      H->mask_tiles = tot;
      H->bytes_used = H->off_tiles + 4ull * tot;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Test hook: rows of the mask as the attention kernels see them.
// ---------------------------------------------------------------------------------------------
__global__ void expand_rows_kernel(const unsigned char* blob, int seq, int head, int row_begin, int nrows, int words,
                                   int causal, uint32_t* __restrict__ out) {
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const DamSeq sq = blob_seqs(blob, H)[seq];
  const int a = blockIdx.x;
  if (a >= nrows) return;
  const int i = row_begin + a;
  uint32_t* o = out + (size_t)a * words;
  for (int w = threadIdx.x; w < words; w += blockDim.x) o[w] = 0u;
  __syncthreads();
  if (i < 0 || i >= sq.S) return;
  const int qb = i / DAM_TILE;
  const int row = head * H->total_qblocks + sq.first_qblock + qb;
  const uint32_t* tile_ptr = reinterpret_cast<const uint32_t*>(blob + H->off_tile_ptr);
  const uint32_t* tiles = reinterpret_cast<const uint32_t*>(blob + H->off_tiles);
  DamHeadBits hb = dam_head_bits(blob, H, sq, head);
  for (uint32_t t = tile_ptr[row] + threadIdx.x; t < tile_ptr[row + 1]; t += blockDim.x) {
    uint32_t e = tiles[t];
    if ((e >> 28) == 0u || (e >> 28) == DAM_KIND_GATHERED) continue;   // padding; gathered tiles are handled below
    int kb = (int)(e & 0x0FFFFFFFu);
    uint4 bits = dam_apply_bits(hb, e >> 28, i, kb, causal);
    if (kb * 4 + 3 < words) {
      atomicOr(&o[kb * 4 + 0], bits.x); atomicOr(&o[kb * 4 + 1], bits.y);
      atomicOr(&o[kb * 4 + 2], bits.z); atomicOr(&o[kb * 4 + 3], bits.w);
    }
  }
  // gathered tiles: together they hold exactly the matched columns, in ascending order, 128 per tile
  const uint32_t r0 = tile_ptr[row], r1 = tile_ptr[row + 1];
  int ngath = 0, ncols = 0;
  for (uint32_t t = r0; t < r1; ++t) {
    uint32_t e = tiles[t];
    if ((e >> 28) != DAM_KIND_GATHERED) break;
    ++ngath;
    ncols += (int)((e >> 16) & 0xFFu) + 1;
  }
  if (ngath) {
    // the first `ncols` set bits of V, as words
    int seen = 0;
    for (int w = 0; w < sq.W && w < words; ++w) {
      uint32_t vw = hb.V[w];
      int pc = __popc(vw);
      if (seen + pc > ncols) {              // keep only the lowest (ncols - seen) set bits
        uint32_t keep = 0u;
        for (int k = 0; k < ncols - seen; ++k) { uint32_t low = vw & (0u - vw); keep |= low; vw ^= low; }
        vw = keep; pc = ncols - seen;
      }
      if (threadIdx.x == 0 && vw) atomicOr(&o[w], vw);
      seen += pc;
      if (seen >= ncols) break;
    }
  }
}

}  // namespace

cudaError_t dam_launch_init_blob(const dam_shape_t* shape, int pcl_max, uint32_t flags, void* blob,
                                 const DamHeader& host_hdr, cudaStream_t st) {
  int mode = (flags & DAM_FLAG_ALL_ONES) ? ((flags & DAM_FLAG_CAUSAL_LIST) ? 1 : 0) : -1;
  init_blob_kernel<<<1, 256, 0, st>>>(reinterpret_cast<unsigned char*>(blob), host_hdr, shape->cu_seqlens_dev,
                                      pcl_max, shape->num_q_heads, mode);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Z-score / min-max (Appendix B): statistics of X = max(P, eps) over all L x L cells of one map (cells above
// the diagonal are eps), in double, one block per map with a fixed reduction order; then the true mask with
// the map's own threshold  X >= eps + tau (std + eps)  or  X >= eps + tau (max - eps + eps).
// ---------------------------------------------------------------------------------------------
struct DamMapStats { double sum, sumsq; float mx; float pad; };

__global__ void __launch_bounds__(1024)
map_stats_kernel(const unsigned char* blob, const float* __restrict__ P, unsigned char* scratch, uint64_t off_cnt, float eps) {
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int sh = blockIdx.x;
  const int b = sh / H->num_q_heads, h = sh % H->num_q_heads;
  const DamSeq sq = blob_seqs(blob, H)[b];
  if (sq.L == 0) return;
  const int L = sq.L;
  const float* Ph = P + sq.p_off + (uint64_t)h * L * L;
  double s = 0.0, s2 = 0.0;
  float mx = eps;
  for (long long idx = threadIdx.x; idx < (long long)L * L; idx += blockDim.x) {
    const int i = (int)(idx / L), j = (int)(idx % L);
    const float x = fmaxf(j <= i ? __ldg(Ph + idx) : 0.f, eps);
    s += (double)x; s2 += (double)x * (double)x;
    mx = fmaxf(mx, x);
  }
  __shared__ double sh_s[1024], sh_s2[1024];
  __shared__ float sh_mx[1024];
  sh_s[threadIdx.x] = s; sh_s2[threadIdx.x] = s2; sh_mx[threadIdx.x] = mx;
  __syncthreads();
  for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) {
      sh_s[threadIdx.x] += sh_s[threadIdx.x + o];
      sh_s2[threadIdx.x] += sh_s2[threadIdx.x + o];
      sh_mx[threadIdx.x] = fmaxf(sh_mx[threadIdx.x], sh_mx[threadIdx.x + o]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    DamMapStats* st = reinterpret_cast<DamMapStats*>(reinterpret_cast<int32_t*>(scratch + off_cnt) + sq.cnt_off +
                                                     (uint64_t)h * dam_cnt_stride(sq.L, sq.W, sq.nL));
    st->sum = sh_s[0]; st->sumsq = sh_s2[0]; st->mx = sh_mx[0]; st->pad = 0.f;
  }
}

__global__ void bits_from_scores_per_map_kernel(unsigned char* blob, const float* __restrict__ P,
                                                const unsigned char* scratch, uint64_t off_cnt, int transform,
                                                float tau_f, float eps_f) {
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int sh = blockIdx.y;
  const int b = sh / H->num_q_heads, h = sh % H->num_q_heads;
  const DamSeq sq = blob_seqs(blob, H)[b];
  if (sq.L == 0) return;
  const DamMapStats st = *reinterpret_cast<const DamMapStats*>(reinterpret_cast<const int32_t*>(scratch + off_cnt) + sq.cnt_off +
                                                               (uint64_t)h * dam_cnt_stride(sq.L, sq.W, sq.nL));
  const double tau = (double)tau_f, eps = (double)eps_f, N = (double)sq.L * (double)sq.L;
  double thr;
  if (transform == DAM_TRANSFORM_ZSCORE) {
    const double mean = st.sum / N;
    const double var = st.sumsq / N - mean * mean;
    thr = eps + tau * (sqrt(var > 0.0 ? var : 0.0) + eps);
  } else {
    thr = eps + tau * (((double)st.mx - eps) + eps);
  }
  uint32_t* M = reinterpret_cast<uint32_t*>(blob + H->off_true) + sq.true_off + (uint64_t)h * sq.L * sq.W;
  const float* Ph = P + sq.p_off + (uint64_t)h * sq.L * sq.L;
  const int lane = threadIdx.x & 31;
  const long long nitems = (long long)sq.L * sq.W;
  const long long wstride = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long it = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); it < nitems; it += wstride) {
    const int i = (int)(it / sq.W), w = (int)(it % sq.W);
    const int j = w * 32 + lane;
    const bool in = j < sq.L && j <= i;
    const float x = fmaxf(in ? __ldg(Ph + (size_t)i * sq.L + j) : 0.0f, eps_f);
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, in && (double)x >= thr);
    if (lane == 0) M[(size_t)i * sq.W + w] = word;
  }
}

cudaError_t dam_launch_bits_from_scores(const float* P, const DamBuildCtx& c, cudaStream_t st) {
  if (c.max_L == 0) return cudaSuccess;
  long long items = (long long)c.max_L * c.max_W;
  int bx = (int)((items + 7) / 8);
  if (bx > 4096) bx = 4096;
  dim3 grid(bx, c.num_seqs * c.Hq);
  if (c.per_map) {
    // the statistics borrow the first bytes of every map's counter area, which is cleared again afterwards
    map_stats_kernel<<<c.num_seqs * c.Hq, 1024, 0, st>>>(c.blob, P, c.scratch, c.off_cnt, c.eps);
    bits_from_scores_per_map_kernel<<<grid, 256, 0, st>>>(c.blob, P, c.scratch, c.off_cnt, c.per_map, c.tau, c.eps);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return cudaMemsetAsync(c.scratch + c.off_cnt, 0, c.off_cnt_end - c.off_cnt, st);
  }
  bits_from_scores_kernel<<<grid, 256, 0, st>>>(c.blob, P, c.pstar);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Multi-sample capture (Sec. 4.2.2): A[h][i][j] += sum over the samples b of a batch of P_b[h][i][j]
// (i, j < L_b = min(S_b, L_max)), C[i] += #{b : L_b > i}.  One thread per cell of a row; the samples
// of the batch are added in index order, so the fp32 sums do not depend on the launch.
// ---------------------------------------------------------------------------------------------
__global__ void capture_accumulate_kernel(const float* __restrict__ P, const int32_t* __restrict__ cu, int num_seqs,
                                          int Hq, int Lmax, float* __restrict__ A, int32_t* __restrict__ C) {
  const int i = blockIdx.x, h = blockIdx.y;
  unsigned long long p_off = 0;                      // fp32 elements before sample b in the score tensor
  int cnt = 0;
  for (int b = 0; b < num_seqs; ++b) {
    const int S = cu[b + 1] - cu[b];
    const int L = S < Lmax ? S : Lmax;
    if (i < L) {
      ++cnt;
      const float* Pr = P + p_off + ((unsigned long long)h * L + i) * L;
      float* Ar = A + ((unsigned long long)h * Lmax + i) * Lmax;
      for (int j = threadIdx.x; j <= i; j += blockDim.x) Ar[j] += __ldg(Pr + j);
    }
    p_off += (unsigned long long)Hq * L * L;
  }
  if (h == 0 && threadIdx.x == 0) C[i] += cnt;
}

// Averaged map in the layout the rule kernels read: for every (sequence b, head h) of the target shape,
// P_out[i][j] = A[h][i][j] / (float(C[i]) + eps) for j <= i < L_b, 0 above the diagonal (IEEE single division).
__global__ void capture_average_kernel(const float* __restrict__ A, const int32_t* __restrict__ C, int Lmax, float eps,
                                       const int32_t* __restrict__ cu, int num_seqs, int Hq, float* __restrict__ P_out) {
  const int i = blockIdx.x, h = blockIdx.y;
  const float den = (float)C[i] + eps;
  const float* Ar = A + ((unsigned long long)h * Lmax + i) * Lmax;
  unsigned long long p_off = 0;
  for (int b = 0; b < num_seqs; ++b) {
    const int S = cu[b + 1] - cu[b];
    const int L = S < Lmax ? S : Lmax;
    if (i < L) {
      float* Pr = P_out + p_off + ((unsigned long long)h * L + i) * L;
      for (int j = threadIdx.x; j < L; j += blockDim.x) Pr[j] = j <= i ? Ar[j] / den : 0.f;
    }
    p_off += (unsigned long long)Hq * L * L;
  }
}

cudaError_t dam_launch_capture_accumulate(const float* P, const dam_shape_t* s, int Lmax, float* A, int32_t* C,
                                          cudaStream_t st) {
  int maxL = 0;
  for (int b = 0; b < s->num_seqs; ++b) {
    int L = s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b];
    L = L < Lmax ? L : Lmax;
    maxL = L > maxL ? L : maxL;
  }
  if (maxL == 0) return cudaSuccess;
  capture_accumulate_kernel<<<dim3(maxL, s->num_q_heads), 256, 0, st>>>(P, s->cu_seqlens_dev, s->num_seqs,
                                                                        s->num_q_heads, Lmax, A, C);
  return cudaGetLastError();
}

cudaError_t dam_launch_capture_average(const float* A, const int32_t* C, int Lmax, float eps, const dam_shape_t* s,
                                       float* P_out, cudaStream_t st) {
  int maxL = 0;
  for (int b = 0; b < s->num_seqs; ++b) {
    int L = s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b];
    L = L < Lmax ? L : Lmax;
    maxL = L > maxL ? L : maxL;
  }
  if (maxL == 0) return cudaSuccess;
  capture_average_kernel<<<dim3(maxL, s->num_q_heads), 256, 0, st>>>(A, C, Lmax, eps, s->cu_seqlens_dev, s->num_seqs,
                                                                     s->num_q_heads, P_out);
  return cudaGetLastError();
}

// The counters of the rule kernels start at zero: counts + prefix + tile popcounts, row counts, histogram,
// cursors.  Enqueued before the kernel that produces the true mask, so that the rule kernels follow it directly.
cudaError_t dam_launch_rule_prepare(const DamBuildCtx& c, cudaStream_t st) {
  // the sections are contiguous (status block and work counter of the scoring kernel | counts | row counts |
  // histogram | cursors): one fill
  return cudaMemsetAsync(c.scratch, 0, c.off_cursor + 4ull * DAM_HIST, st);
}

cudaError_t dam_launch_rule(const DamBuildCtx& c, cudaStream_t st) {
  cudaError_t e;
  if (c.max_nL > 0) {
    dim3 g(c.max_nL * (c.max_nL + 1) / 2, c.num_seqs * c.Hq);
    if ((e = launch_chained(counts_kernel, g, dim3(DAM_TILE), st, c.blob, c.scratch, c.off_cnt)) != cudaSuccess) return e;
    if ((e = launch_chained(match_kernel, dim3(c.num_seqs * c.Hq), dim3(1024), st, c.blob, c.scratch, c.off_cnt, c.mu,
                            c.min_support)) != cudaSuccess) return e;
  }
  if (c.rows > 0) {
    int blocks = (c.prows + 7) / 8;
    if ((e = launch_chained(classify_kernel, dim3(blocks), dim3(256), st, c.blob, c.scratch, c.off_cnt, c.off_items,
                            c.off_rowcnt)) != cudaSuccess) return e;
    if ((e = launch_chained(order_kernel, dim3((c.prows + 1023) / 1024), dim3(1024), st, c.blob, c.scratch, c.off_items,
                            c.off_rowcnt)) != cudaSuccess)
      return e;
  }
  return cudaGetLastError();
}

cudaError_t dam_launch_all_ones(const dam_shape_t* shape, int causal, void* blob, cudaStream_t st) {
  int rows = 0;
  for (int b = 0; b < shape->num_seqs; ++b)
    rows += (shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b] + DAM_TILE - 1) / DAM_TILE;
  rows *= shape->num_q_heads;
  if (rows == 0) return cudaSuccess;
  all_ones_kernel<<<(rows + 7) / 8, 256, 0, st>>>(reinterpret_cast<unsigned char*>(blob), causal);
  return cudaGetLastError();
}

// Active cells of the S x S mask of every (sequence, head): the true mask inside the window; below it every row
// keeps the matched columns and the matched diagonals, and a cell that is both (key j = i - r with V[j] and D[r],
// possible on rows L .. 2L-2 only) counts once (Sec. 4.3, Case 2).  One block per (sequence, head); integer
// arithmetic, the block's partial sums are added in a fixed order.
__global__ void __launch_bounds__(256)
active_elems_kernel(const unsigned char* blob, unsigned long long* __restrict__ out) {
  const DamHeader* H = reinterpret_cast<const DamHeader*>(blob);
  const int b = blockIdx.x / H->num_q_heads, h = blockIdx.x % H->num_q_heads;
  const DamSeq sq = blob_seqs(blob, H)[b];
  __shared__ unsigned long long part[256];
  unsigned long long n = 0;
  if (sq.L > 0) {
    const DamHeadBits hb = dam_head_bits(blob, H, sq, h);
    const size_t words = (size_t)sq.L * sq.W;
    for (size_t w = threadIdx.x; w < words; w += blockDim.x) n += (unsigned long long)__popc(__ldg(hb.M + w));
    if (sq.S > sq.L) {
      // rows i in [L, min(S, 2L-1)): overlap(i) = #{j < L : V[j] and D[i-j]}; keys j .. j+31 read Drev bits from L-1-i+j
      const int i_end = sq.S < 2 * sq.L - 1 ? sq.S : 2 * sq.L - 1;
      long long both = 0;
      for (int i = sq.L + (int)threadIdx.x; i < i_end; i += blockDim.x)
        for (int w = 0; w < sq.W; ++w) {
          const uint32_t v = __ldg(hb.V + w);
          if (v) both += __popc(v & dam_window32(hb.Drev, sq.W, sq.L - 1 - i + 32 * w));
        }
      if (threadIdx.x == 0) {
        long long pd = 0, pv = 0;
        for (int w = 0; w < sq.W; ++w) { pd += __popc(__ldg(hb.D + w)); pv += __popc(__ldg(hb.V + w)); }
        n += (unsigned long long)((long long)(sq.S - sq.L) * (pd + pv));
      }
      n -= (unsigned long long)both;      // (modular arithmetic: the block's total is what counts)
    }
  }
  part[threadIdx.x] = n;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int k = 0; k < 256; ++k) t += part[k];
    out[blockIdx.x] = t;
  }
}

cudaError_t dam_launch_active_elems(const void* blob, int num_seqs, int Hq, unsigned long long* out, cudaStream_t st) {
  active_elems_kernel<<<num_seqs * Hq, 256, 0, st>>>(reinterpret_cast<const unsigned char*>(blob), out);
  return cudaGetLastError();
}

cudaError_t dam_launch_expand_rows(const void* blob, int seq, int head, int row_begin, int nrows, int words,
                                   int causal, uint32_t* out, cudaStream_t st) {
  expand_rows_kernel<<<nrows, 128, 0, st>>>(reinterpret_cast<const unsigned char*>(blob), seq, head, row_begin, nrows,
                                            words, causal, out);
  return cudaGetLastError();
}
