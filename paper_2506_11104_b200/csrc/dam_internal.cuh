// Internal layout of the mask blob and device helpers shared by the DAM kernels.
//
// The blob is one flat, relocatable buffer (byte offsets from its start, little endian):
//
//   DamHeader (256 B)            magic, status word, counts, section offsets
//   DamSeq[num_seqs]             per sequence: token start, S, L = min(S, pcl_max), q-block range,
//                                word offsets of its bit sections
//   qb_seq[total_qblocks]        sequence index of every global 128-row query block
//   per (seq, head) pattern bits 3 * W words: D (matched diagonal offsets r), Drev (D reversed:
//                                bit x = D[L-1-x]), V (matched columns c); W = ceil(L/32) rounded
//                                up to a multiple of 4 words
//   per (seq, head) true mask    L rows x W words, bit (j % 32) of word (j / 32) = M[i][j]
//   pair_tab[total_pairs]        first global q-block of every pair of adjacent q-blocks (2p, 2p+1) of a
//                                sequence; bit 31 set when the second block exists
//   tile_ptr[rows + 1]           start of every row's entries in tiles[], rows = head * total_qblocks + global
//                                q-block.  Every pair of adjacent q-blocks owns a fixed range of tiles[] (the sum
//                                of the two rows' upper bounds, known from the shapes alone): the first row's
//                                entries, directly followed by the second row's, then zero entries (kind 0) up to
//                                the next pair.  [tile_ptr[r], tile_ptr[r + 1]) therefore holds row r's entries
//                                and possibly zero entries behind them, which every reader skips.
//   items[prows]                 work list of the attention kernel (DamItem, 32 B): one entry per
//                                (head, pair), the pair with the most listed tiles (both blocks
//                                together) first, with everything a CTA needs to start on it
//   tiles[...]                   one u32 per listed tile: kv tile index | kind << 28
//
// A PARTIAL tile stores no bits of its own: inside the window they are the true-mask words of the
// row, below it they follow from V and Drev (Sec. 4.3, Case 2), see dam_tile_row_bits.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dam.h"

#define DAM_TILE 128
#define DAM_MAGIC 0x4B4D4144u      /* "DAMK" */
#define DAM_KIND_FULL 1u
#define DAM_KIND_PARTIAL 2u
#define DAM_KIND_GATHERED 3u    /* entry = gathered tile index | (columns in it - 1) << 16 | kind << 28 */
#define DAM_FLAG_ALL_ONES 1u
#define DAM_FLAG_CAUSAL_LIST 2u    /* tile lists hold only kb <= qb */
#define DAM_FLAG_GATHER 4u         /* rows from 2L-1 on list gathered-column tiles instead of vertical tiles */
#define DAM_HIST 4096

struct DamHeader {
  uint32_t magic;
  uint32_t status;          // device-side dam_status_t, 0 = ok
  uint32_t version;
  uint32_t flags;
  int32_t num_seqs;
  int32_t num_q_heads;
  int32_t total_qblocks;
  int32_t rows;             // num_q_heads * total_qblocks
  uint32_t tile_capacity;   // entries that fit in tiles[]
  uint32_t total_tiles;     // entries in use
  uint32_t full_tiles;
  uint32_t pcl_max;
  uint64_t off_seq, off_qbseq, off_dv, off_true, off_tile_ptr, off_work, off_tiles;
  uint64_t bytes_used;
  uint64_t causal_tiles;    // sum over heads and sequences of nq (nq + 1) / 2
  uint64_t off_pairtab;
  int32_t total_pairs;      // sum over sequences of ceil(nq / 2)
  int32_t prows;            // num_q_heads * total_pairs
  uint64_t gath_tiles;      // gathered-column tiles over all (seq, head): sum Hq * nL (capacity, 128 keys each)
  uint64_t attn_scratch_bytes;   // scratch dam_sparse_attention needs for this blob
  uint64_t mask_tiles;      // 128 x 128 tiles of the masks that hold an active cell (= total_tiles unless gathered)
  uint64_t head_tile_cap;   // entries of tiles[] every head owns (sum of the row bounds of all sequences)
  uint64_t reserved[11];    // [0]: 1 when the window map was scored by the tensor-core kernel (test hook)
};
static_assert(sizeof(DamHeader) == 256, "DamHeader must be 256 bytes");

struct DamItem {            // one unit of attention work: query blocks (2p, 2p+1) of one (sequence, head)
  int32_t head, tok0, qb0, S;      // tok0 = first token of the sequence, qb0 = 2p, S = sequence length
  uint32_t a0, a1, b1;             // tile list [a0, a1) of block 2p and [a1, b1) of block 2p+1
  uint32_t seq_hasB;               // sequence index | (second block exists) << 31
};
static_assert(sizeof(DamItem) == 32, "DamItem must be 32 bytes");

struct DamSeq {
  int32_t tok_start, S, L, nq;
  int32_t first_qblock, W, nL, first_pair;
  uint64_t dv_off;     // u32 words from off_dv: head h at dv_off + h * 3 * W
  uint64_t true_off;   // u32 words from off_true: head h at true_off + h * L * W
  uint64_t p_off;      // fp32 elements into a score tensor: head h at p_off + h * L * L
  uint64_t cnt_off;    // int32 elements into the build scratch count area: head h at cnt_off + h * cnt_stride
  uint64_t gath_off;   // gathered-column tiles: head h owns tiles [gath_off + h * nL, +nL)
  uint64_t tile_base;  // first entry of the sequence's rows inside a head's range of tiles[]
};
static_assert(sizeof(DamSeq) == 80, "DamSeq must be 80 bytes");

// Per-(seq, head) words in the build scratch count area:
//   cntD[L], cntV[L], prefD[W + 1], prefV[W + 1], tile_pop[nL * nL], padded to a multiple of 4.
__host__ __device__ inline uint64_t dam_cnt_stride(int L, int W, int nL) {
  uint64_t n = 2ull * L + 2ull * (W + 1) + (uint64_t)nL * nL;
  return (n + 3) & ~3ull;
}
__host__ __device__ inline int dam_words(int L) { return (((L + 31) >> 5) + 3) & ~3; }
__host__ __device__ inline uint64_t dam_align(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// Upper bound on listed tiles of one q-block row of a DAM mask (see dam_mask_sizes): the window's column
// tiles plus the diagonal band, never more than the causal tiles of the row.  A row served by gathered-column
// tiles lists at most nL gathered tiles plus the band tiles [qb - nL, qb].
__host__ __device__ inline int dam_row_tile_bound(int qb, int nL, int L, int gather) {
  const int gather_first = (2 * L - 1 + DAM_TILE - 1) / DAM_TILE;
  if (gather && L > 0 && qb >= gather_first) {
    const int band = qb + 1 < nL + 1 ? qb + 1 : nL + 1;
    return nL + band;
  }
  int a = qb + 1, b = 2 * nL + 1;
  return a < b ? a : b;
}

// Sum of dam_row_tile_bound over the query blocks 0 .. qb-1 of a sequence: where block qb's entries start inside
// the sequence's range of a head.  (From the first gathered block on every bound is 2 nL + 1: nL gathered tiles
// and the nL + 1 band tiles; before it, min(q + 1, 2 nL + 1).)
__host__ __device__ inline uint64_t dam_row_tile_prefix(int qb, int nL, int L, int gather) {
  const int gather_first = (2 * L - 1 + DAM_TILE - 1) / DAM_TILE;
  const uint64_t m = 2ull * nL + 1;
  const uint64_t k = (gather && L > 0 && qb > gather_first) ? (uint64_t)gather_first : (uint64_t)qb;   // blocks on the plain rule
  const uint64_t j = k < m ? k : m;
  return j * (j + 1) / 2 + (k - j) * m + ((uint64_t)qb - k) * m;
}

// Gathered-column tiles serve the query blocks that start at or after row 2L - 1 (first multiple of 128).
__host__ __device__ inline int dam_gather_first_qblock(int L) { return (2 * L - 1 + DAM_TILE - 1) / DAM_TILE; }
__host__ __device__ inline int dam_gather_first_row(int L) { return dam_gather_first_qblock(L) * DAM_TILE; }

struct DamHeadBits {
  const uint32_t* D;
  const uint32_t* Drev;
  const uint32_t* V;
  const uint32_t* M;
  int L, W, S;
  int gather_from;     // first row whose matched columns are served by gathered tiles (INT_MAX: none)
};

__device__ __forceinline__ DamHeadBits dam_head_bits(const unsigned char* blob, const DamHeader* hdr,
                                                     const DamSeq& sq, int head) {
  DamHeadBits hb;
  const uint32_t* dv = reinterpret_cast<const uint32_t*>(blob + hdr->off_dv) + sq.dv_off + (uint64_t)head * 3 * sq.W;
  hb.D = dv;
  hb.Drev = dv + sq.W;
  hb.V = dv + 2 * sq.W;
  hb.M = reinterpret_cast<const uint32_t*>(blob + hdr->off_true) + sq.true_off + (uint64_t)head * sq.L * sq.W;
  hb.L = sq.L;
  hb.W = sq.W;
  hb.S = sq.S;
  hb.gather_from = (hdr->flags & DAM_FLAG_GATHER) ? dam_gather_first_row(sq.L) : 0x7FFFFFFF;
  return hb;
}

// bits [x, x + 32) of a bit array of nwords words; zero outside the array. x may be negative.
__device__ __forceinline__ uint32_t dam_window32(const uint32_t* __restrict__ bits, int nwords, int x) {
  int w = x >> 5;  // arithmetic shift: floor
  int sh = x & 31;
  uint32_t lo = (w >= 0 && w < nwords) ? __ldg(bits + w) : 0u;
  uint32_t hi = (w + 1 >= 0 && w + 1 < nwords) ? __ldg(bits + w + 1) : 0u;
  return __funnelshift_r(lo, hi, sh);
}

// The 128 mask bits of row i (index inside the sequence) against kv tile kb of a PARTIAL tile.
// Inside the window (i < L): the true-mask words.  Below it: matched columns of this tile OR the
// matched diagonals, key j active iff D[i - j]; with Drev[x] = D[L-1-x] the keys j0 .. j0+127 read
// Drev bits x0 .. x0+127, x0 = L - 1 - i + j0 (ascending in j), which also excludes j > i.
__device__ __forceinline__ uint4 dam_tile_row_bits(const DamHeadBits& hb, int i, int kb) {
  uint4 r = make_uint4(0u, 0u, 0u, 0u);
  const int j0 = kb * DAM_TILE;
  if (i >= hb.S) return r;
  if (i < hb.L) {
    if (j0 < hb.L) r = __ldg(reinterpret_cast<const uint4*>(hb.M + (size_t)i * hb.W + kb * 4));
  } else {
    if (j0 < hb.L && i < hb.gather_from) r = __ldg(reinterpret_cast<const uint4*>(hb.V + kb * 4));
    const int x0 = hb.L - 1 - i + j0;
    if (x0 + DAM_TILE > 0 && x0 < hb.L) {
      r.x |= dam_window32(hb.Drev, hb.W, x0);
      r.y |= dam_window32(hb.Drev, hb.W, x0 + 32);
      r.z |= dam_window32(hb.Drev, hb.W, x0 + 64);
      r.w |= dam_window32(hb.Drev, hb.W, x0 + 96);
    }
  }
  return r;
}

// ones for t in [0, n), n clipped to [0, 128]
__device__ __forceinline__ uint4 dam_low_ones128(int n) {
  uint4 r;
  auto w = [](int k) -> uint32_t { return k >= 32 ? 0xFFFFFFFFu : (k <= 0 ? 0u : ((1u << k) - 1u)); };
  r.x = w(n);
  r.y = w(n - 32);
  r.z = w(n - 64);
  r.w = w(n - 96);
  return r;
}

// Final 128 bits the attention kernels apply for row i against tile kb.
__device__ __forceinline__ uint4 dam_apply_bits(const DamHeadBits& hb, uint32_t kind, int i, int kb, int causal) {
  uint4 b = (kind == DAM_KIND_FULL) ? make_uint4(~0u, ~0u, ~0u, ~0u) : dam_tile_row_bits(hb, i, kb);
  const int j0 = kb * DAM_TILE;
  if (i >= hb.S) return make_uint4(0u, 0u, 0u, 0u);
  int n = hb.S - j0;                       // keys beyond the sequence end do not exist
  if (causal) { int c = i - j0 + 1; n = c < n ? c : n; }
  if (n < DAM_TILE) {
    uint4 m = dam_low_ones128(n);
    b.x &= m.x; b.y &= m.y; b.z &= m.z; b.w &= m.w;
  }
  return b;
}

// ---- per-device state ---------------------------------------------------------------------------
// What a launch needs to know about the device it runs on, and the one-off set-up steps that CUDA wants per
// device (cudaFuncSetAttribute for the large dynamic shared memory of the tensor-core kernels).  Records are kept
// per device ordinal and filled on first use under a mutex, so that one process may drive several GPUs from
// several threads.
struct DamDeviceInfo { int cc_major, sm_count, smem_optin; };
typedef cudaError_t (*dam_device_query_fn)(int device, DamDeviceInfo* out);
typedef cudaError_t (*dam_device_setup_fn)(void);

class DamDeviceTable {
 public:
  static constexpr int kMaxDevices = 64;
  static constexpr int kMaxSetups = 8;
  // The record of `device`, filled by `query` the first time the ordinal is seen.
  cudaError_t info(int device, dam_device_query_fn query, DamDeviceInfo* out);
  // Runs `fn` (with `device` current) unless set-up step `key` already succeeded on that device.
  cudaError_t once(int device, int key, dam_device_setup_fn fn);
 private:
  struct Slot { bool filled; DamDeviceInfo info; bool done[kMaxSetups]; };
  Slot slots_[kMaxDevices] = {};
};
enum { DAM_SETUP_ATTN_SMEM = 0, DAM_SETUP_SCORE_SMEM = 1, DAM_SETUP_DECODE_SMEM = 2 };

DamDeviceTable& dam_device_table();                                       // the library's own table
cudaError_t dam_current_device(int* device, DamDeviceInfo* info);         // ordinal and record of the current device

// ---- host-side launch entry points of the kernel files -----------------------------------------
struct DamBuildCtx {
  unsigned char* blob;
  unsigned char* scratch;
  int num_seqs, Hq, Hkv, d, dtype;
  int total_qblocks, rows, prows;
  int max_L, max_W, max_nL, max_nq;
  float pstar;       // single-compare threshold on p equivalent to the Box-Cox chain
  int per_map;       // 0, or the dam_transform_t whose threshold depends on each map's own statistics
  float tau, eps;    // for the per-map thresholds
  float mu;
  int min_support;
  float scale;
  int gather;        // list gathered-column tiles
  uint64_t off_cnt, off_cnt_end, off_rowcnt, off_hist, off_cursor, off_items;   // scratch sections
  uint64_t off_true, true_bytes;                                     // true-mask section of the blob
};

cudaError_t dam_launch_init_blob(const dam_shape_t* shape, int pcl_max, uint32_t flags, void* blob,
                                 const DamHeader& host_hdr, cudaStream_t st);
cudaError_t dam_launch_scores_ref(const void* Q, const void* K, const dam_shape_t* shape, const DamBuildCtx& c,
                                  float* scores_dump, cudaStream_t st);
cudaError_t dam_launch_bits_from_scores(const float* P, const DamBuildCtx& c, cudaStream_t st);
cudaError_t dam_launch_rule_prepare(const DamBuildCtx& c, cudaStream_t st);   // before the true mask is produced
cudaError_t dam_launch_rule(const DamBuildCtx& c, cudaStream_t st);
cudaError_t dam_launch_all_ones(const dam_shape_t* shape, int causal, void* blob, cudaStream_t st);
cudaError_t dam_launch_expand_rows(const void* blob, int seq, int head, int row_begin, int nrows, int words,
                                   int causal, uint32_t* out, cudaStream_t st);
cudaError_t dam_launch_active_elems(const void* blob, int num_seqs, int Hq, unsigned long long* out, cudaStream_t st);
// `ranges` (device, int32[2 * num_seqs], or NULL): only the pairs of query blocks whose first row lies in
// [ranges[2b], ranges[2b+1]) of sequence b are computed
cudaError_t dam_launch_attn_ref(const void* Q, const void* K, const void* V, const void* blob,
                                const dam_shape_t* shape, int causal, float scale, void* O, float* lse,
                                void* scratch, const int32_t* ranges, cudaStream_t st);
// tensor-core paths (bf16, d = 128); return cudaErrorNotSupported when the shape does not qualify
cudaError_t dam_launch_attn_sm100(const void* Q, const void* K, const void* V, const void* blob,
                                  const dam_shape_t* shape, int causal, float scale, void* O, float* lse,
                                  void* scratch, size_t scratch_bytes, const int32_t* ranges, bool run_gather, cudaStream_t st);
cudaError_t dam_launch_scores_sm100(const void* Q, const void* K, const dam_shape_t* shape, const DamBuildCtx& c,
                                    float* scores_dump, cudaStream_t st);

cudaError_t dam_launch_capture_accumulate(const float* P, const dam_shape_t* shape, int Lmax, float* A, int32_t* C,
                                          cudaStream_t st);
cudaError_t dam_launch_capture_average(const float* A, const int32_t* C, int Lmax, float eps, const dam_shape_t* shape,
                                       float* P_out, cudaStream_t st);
cudaError_t dam_launch_decode_group(const void* q, const void* K, const void* V, const void* blob, const dam_shape_t* shape,
                                    const int32_t* pos_dev, float scale, void* O, float* lse, void* scratch, cudaStream_t st);
cudaError_t dam_launch_decode(const void* q, const void* K, const void* V, const void* blob, const dam_shape_t* shape,
                              const int32_t* pos_dev, float scale, void* O, float* lse, void* scratch, cudaStream_t st);

cudaError_t dam_launch_bounded_wait_selftest(void* scratch, unsigned long long limit_ns, cudaStream_t st);
