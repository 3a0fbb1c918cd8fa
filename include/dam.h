/*
 * dam.h -- C ABI of the B200 (sm_100a) library for long-context prefill attention under
 * Dynamic Attention Masks (DAM, arXiv 2506.11104).
 *
 * Two stages, one call each:
 *
 *   dam_build_masks       builds, for every (sequence, query head), the true mask over the
 *                         pattern-capture window and the matched diagonal / vertical patterns,
 *                         and writes them with a tile list into one compact mask blob
 *                         (paper Sec. 4.2.1 - 4.2.4, Sec. 4.3 "Case 1 / Case 2");
 *   dam_sparse_attention  computes softmax(Q K^T / sqrt(d) with masked logits = -inf) V, visiting
 *                         only the 128 x 128 tiles the blob lists (paper Sec. 3 and Sec. 4.3, last
 *                         paragraph).
 *
 * Conventions that hold for every entry point
 *   - plain C types only; "device" pointers are CUDA global-memory pointers on the current device,
 *     "host" pointers are ordinary host memory; `stream` is a cudaStream_t passed as void*;
 *   - the caller owns every buffer; the library allocates no device memory, keeps no pointer after
 *     the enqueued work retires, and enqueues all work on `stream` without synchronising it
 *     (exceptions are stated at the function);
 *   - every function returns a dam_status_t; argument errors are detected on the host before
 *     anything is enqueued and nothing is written in that case;
 *   - problems only the device can see (a bounded wait that expired, an attention scratch that is too
 *     small for the blob it is used with) are recorded in the status word at the start of the mask blob / attention
 *     scratch and are read back with dam_poll_status;
 *   - layouts: Q, O are [total_tokens, num_q_heads, head_dim]; K, V are
 *     [total_tokens, num_kv_heads, head_dim]; sequences are packed back to back (token-major) and
 *     delimited by cu_seqlens[num_seqs + 1]; strides are given in elements and head_dim is
 *     contiguous; LSE is [num_q_heads, total_tokens] float;
 *   - query head h reads K, V of KV head h / (num_q_heads / num_kv_heads).
 */
#ifndef DAM_H_
#define DAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dam_status_t {
  DAM_OK = 0,
  DAM_ERR_INVALID_ARGUMENT = 1, /* null / misaligned pointer, inconsistent shape, bad rule value   */
  DAM_ERR_UNSUPPORTED = 2,      /* valid request this build has no kernel for                      */
  DAM_ERR_BUFFER_TOO_SMALL = 3, /* mask blob or scratch smaller than dam_mask_sizes reports        */
  DAM_ERR_CUDA = 4,             /* a CUDA runtime / driver call failed                             */
  DAM_ERR_DEVICE_TIMEOUT = 5,   /* a bounded wait inside a kernel expired (kernel returned early)  */
  DAM_ERR_INTERNAL = 6
} dam_status_t;

typedef enum dam_dtype_t { DAM_BF16 = 0, DAM_F32 = 1 } dam_dtype_t;

/* Shapes of one layer's attention call. */
typedef struct dam_shape_t {
  uint32_t struct_size;           /* sizeof(dam_shape_t), for ABI checking                          */
  int32_t num_seqs;               /* B >= 1                                                        */
  const int32_t* cu_seqlens_host; /* HOST, B + 1 entries, [0] = 0, non-decreasing                   */
  const int32_t* cu_seqlens_dev;  /* DEVICE, same values                                            */
  int32_t total_tokens;           /* = cu_seqlens[B]                                                */
  int32_t max_seqlen;             /* >= every sequence length                                       */
  int32_t num_q_heads;            /* Hq                                                             */
  int32_t num_kv_heads;           /* Hkv, Hq % Hkv == 0                                             */
  int32_t head_dim;               /* d; multiple of 8, <= 256 (tensor-core path: bf16, d = 128 or 64) */
  int32_t dtype;                  /* dam_dtype_t of Q, K, V, O                                      */
  int64_t q_stride_tok, q_stride_head; /* elements                                                  */
  int64_t k_stride_tok, k_stride_head;
  int64_t v_stride_tok, v_stride_head;
  int64_t o_stride_tok, o_stride_head;
} dam_shape_t;

/* Mask-rule parameters (paper Sec. 4.2; the paper's runs use PCL 512, tau 0.3, mu 0.8,
 * lambda 0.5, eps 1e-8). */
typedef struct dam_rule_t {
  uint32_t struct_size; /* sizeof(dam_rule_t)                                                      */
  int32_t pcl_max;      /* L_max >= 1; per sequence L = min(S, L_max) (Sec. 4.2.1)                  */
  float tau;            /* true-mask threshold on the amplified map, > 0 (Sec. 4.2.3)              */
  float mu;             /* pattern match threshold, gamma >= mu (Sec. 4.2.4)                       */
  float lambda;         /* lambda of Box-Cox / Yeo-Johnson (Sec. 4.2.2; the paper uses 0.5)         */
  float eps;            /* clamp constant, > 0 (Sec. 4.2.2)                                        */
  float softmax_scale;  /* 0 selects 1 / sqrt(head_dim) (Sec. 3)                                   */
  int32_t min_support;  /* ignore patterns with fewer cells; 1 = the paper's rule                  */
  uint32_t flags;       /* 0 or DAM_RULE_GATHER_COLUMNS                                            */
  int32_t transform;    /* dam_transform_t: how the map is amplified before tau is applied          */
} dam_rule_t;

/*
 * Amplification applied to X = max(map, eps) before the threshold (Appendix B lists nine; the paper settles on
 * Box-Cox with lambda = 0.5). Each of these is increasing in X and the map is 0 above the diagonal, so the
 * minimum that is subtracted is f(eps) and the true mask is {f(X) - f(eps) >= tau} = {map >= p*}:
 *   BOXCOX      (X^lambda - 1) / lambda, log X for lambda = 0
 *   LOG         log X                        SQRT     sqrt X            ARCSINH   asinh X
 *   YEO_JOHNSON ((X + 1)^lambda - 1) / lambda, log(X + 1) for lambda = 0   (X >= 0 always holds here)
 *   AVERAGE     X itself
 * BOXCOX with lambda = 0.5 is decided by a chain of IEEE single operations (so that two implementations can
 * agree bit for bit: x = max(p, eps); b = (sqrt(x) - 1) * 2; a = b - (sqrt(eps) - 1) * 2; a >= tau); every
 * other case is decided in double precision on the fp32 map value, with tau, eps, lambda widened from float.
 * ZSCORE and MINMAX normalise each map by its own statistics over all L x L cells of X (cells above the diagonal
 * count as eps): (X - mean) / (std + eps) with the population deviation, and (X - min) / (max - min + eps). After
 * the minimum is subtracted they read (X - eps) / (std + eps) >= tau and (X - eps) / (max - eps + eps) >= tau, a
 * threshold per map, decided in double precision. They need a pass over the finished map:
 * dam_build_masks_from_scores offers them, and dam_build_masks does when it is given a scores_dump buffer (the
 * map is written there and thresholded from there; without the buffer it returns UNSUPPORTED).
 *   SUM         the raw sum of Appendix B (method 1): the map handed in is used as it is, like AVERAGE. With one
 *               input the sum is the map itself; with several, pass the accumulated A of dam_capture_accumulate
 *               (not divided by the counts) to dam_build_masks_from_scores.
 */
typedef enum dam_transform_t {
  DAM_TRANSFORM_BOXCOX = 0,
  DAM_TRANSFORM_LOG = 1,
  DAM_TRANSFORM_SQRT = 2,
  DAM_TRANSFORM_ARCSINH = 3,
  DAM_TRANSFORM_YEO_JOHNSON = 4,
  DAM_TRANSFORM_AVERAGE = 5,
  DAM_TRANSFORM_ZSCORE = 6,
  DAM_TRANSFORM_MINMAX = 7,
  DAM_TRANSFORM_SUM = 8
} dam_transform_t;

/*
 * dam_rule_t.flags bit: below row 2L - 1 of a sequence the matched columns (all < L) and the matched
 * diagonals (keys > i - L >= L - 1) never meet (Sec. 4.3, Case 2), so the K / V rows of the matched columns
 * can be copied once per (sequence, head) into dense tiles of 128 keys that every such query block
 * visits as fully active tiles, instead of one mostly-empty tile per stripe. The mask content is
 * unchanged; only the tile lists differ, and dam_sparse_attention needs the larger scratch that
 * dam_mask_sizes then reports. Honoured for the tensor-core shapes (bf16, head_dim 128 or 64); ignored otherwise.
 */
#define DAM_RULE_GATHER_COLUMNS 1u

/* Library version (major * 1000 + minor). No arguments, no device work. */
int32_t dam_version(void);

/* Static text for a status code. Never NULL. */
const char* dam_status_string(dam_status_t status);

/*
 * Sizes of the caller-allocated buffers for one shape.
 *   rule != NULL : blob built by dam_build_masks / dam_build_masks_from_scores. The bound is the
 *                  true-mask bits plus, per 128-row query block, at most 2 * ceil(L / 128) + 1 tile
 *                  entries (a row below the window can only reach the window's columns and the
 *                  L diagonals next to it: Sec. 4.3, Case 2).
 *   rule == NULL : blob built by dam_mask_all_ones (`causal` selects lower-triangular or full).
 * Outputs (HOST pointers, each may be NULL): bytes of the mask blob, of the scratch that the two
 * build calls need, and of the scratch dam_sparse_attention needs. Host only; no device work.
 */
dam_status_t dam_mask_sizes(const dam_shape_t* shape, const dam_rule_t* rule, int32_t causal,
                            size_t* mask_bytes, size_t* build_scratch_bytes,
                            size_t* attn_scratch_bytes);

/*
 * Stage 1 (Sec. 4.2.1 - 4.2.4, 4.3). For every sequence b and query head h:
 *   window = first L_b = min(S_b, pcl_max) tokens; P = causal softmax(Q K^T * scale) over it (fp32);
 *   true mask  M[i][j] = [2 (sqrt(max(P, eps)) - sqrt(eps)) >= tau]   (Box-Cox with lambda = 0.5,
 *   shifted by its minimum, which is the constant B(eps));
 *   cntD[r] = #{i : M[i][i-r]}, cntV[c] = #{i : M[i][c]};  D[r] = [cntD[r] >= mu * (L-r)], same for
 *   V[c], evaluated as one fp32 multiply and compare;  then every 128 x 128 tile of the S_b x S_b
 *   mask (rows below the window follow the matched diagonals / columns) is classified and the
 *   non-empty ones are listed.
 * Q, K: DEVICE, layouts and strides from `shape` (V strides ignored). 16-byte aligned.
 * mask: DEVICE, >= mask_bytes from dam_mask_sizes, 256-byte aligned; fully overwritten.
 * scratch: DEVICE, >= build_scratch_bytes, 256-byte aligned; contents undefined afterwards.
 * scores_dump: DEVICE or NULL. When given, receives P as fp32, for (b, h) at element offset
 *   sum_{b' < b} Hq * L_b'^2 + h * L_b^2, row-major [L_b][L_b], zeros above the diagonal. The mask
 *   decisions are taken on exactly these fp32 values.
 * Errors: INVALID_ARGUMENT (null pointers, alignment, Hq % Hkv, tau <= 0, eps <= 0, pcl_max < 1,
 *   bad cu_seqlens, struct sizes, unknown transform, non-finite lambda), UNSUPPORTED (head_dim),
 *   BUFFER_TOO_SMALL, CUDA.
 */
dam_status_t dam_build_masks(const void* Q, const void* K, const dam_shape_t* shape,
                             const dam_rule_t* rule, void* mask, size_t mask_capacity,
                             void* scratch, size_t scratch_bytes, float* scores_dump,
                             void* stream);

/*
 * Stage 1 without the scoring pass: the rule of Sec. 4.2.2 - 4.3 applied to a caller-supplied fp32
 * map P (DEVICE, same layout as scores_dump above; need not be a softmax). Used to compare masks
 * bit for bit from one shared score tensor. Other arguments and errors as dam_build_masks.
 */
dam_status_t dam_build_masks_from_scores(const float* P, const dam_shape_t* shape,
                                         const dam_rule_t* rule, void* mask, size_t mask_capacity,
                                         void* scratch, size_t scratch_bytes, void* stream);

/*
 * A mask blob that lists every tile (lower-triangular tiles when causal != 0, all tiles otherwise)
 * as fully active: dam_sparse_attention on it is dense attention. Serves as the dense baseline
 * and as a test of the attention kernel alone. The paper has no counterpart (its masks are never
 * all-ones); Sec. 3 defines the dense attention this reproduces.
 * mask: DEVICE, >= mask_bytes from dam_mask_sizes(shape, NULL, causal, ...), 256-byte aligned.
 */
dam_status_t dam_mask_all_ones(const dam_shape_t* shape, int32_t causal, void* mask,
                               size_t mask_capacity, void* stream);

/*
 * Stage 2 (Sec. 3; Sec. 4.3 last paragraph): O = softmax(S') V with S' = Q K^T * scale and
 * S'[i][j] = -inf where the mask is 0 (and where j > i when causal != 0); LSE[h][t] = natural-log
 * sum-exp of row t's active logits. A row with no active key gives O = 0, LSE = -inf.
 * Q, K, V: DEVICE (16-byte aligned); mask: DEVICE blob from a build call or dam_mask_all_ones for the
 * same shape; O: DEVICE, written for every token and head; lse: DEVICE float [Hq][total_tokens].
 * gqa_group must equal num_q_heads / num_kv_heads; softmax_scale 0 selects 1 / sqrt(head_dim).
 * scratch: DEVICE, >= attn_scratch_bytes, 256-byte aligned; it begins with a status word.
 * Tensor-core path (tcgen05 + TMA): dtype bf16, head_dim 128 or 64, 16-byte aligned strides; other
 * shapes run a plain CUDA-core kernel. (Word 4 of the scratch block, i.e. bytes 16..19, is 1 after a call the
 * tensor-core kernel served and 0 otherwise: a hook for tests.)
 * Errors: INVALID_ARGUMENT, UNSUPPORTED, BUFFER_TOO_SMALL, CUDA; DEVICE_TIMEOUT via the status word.
 */
dam_status_t dam_sparse_attention(const void* Q, const void* K, const void* V, const void* mask,
                                  const dam_shape_t* shape, int32_t causal, int32_t gqa_group,
                                  float softmax_scale, void* O, float* lse, void* scratch,
                                  size_t scratch_bytes, void* stream);

/*
 * Multi-sample capture (Sec. 4.2.2: the attention map of a head is the average of the maps of several
 * inputs, A accumulated attention, C valid-token count, A_bar = A / (C + eps)).
 *
 * dam_capture_accumulate adds one batch of samples: P is the fp32 window maps of the batch in the layout of
 * dam_build_masks' scores_dump for `shape` (sample b: [Hq][L_b][L_b], L_b = min(S_b, pcl_max));
 *   A[h][i][j] += sum_b P_b[h][i][j]   (fp32, samples added in index order; j <= i < L_b)
 *   C[i]       += #{b : L_b > i}       (the count depends on the row only: a pair (i, j <= i) is valid in a
 *                                       sample exactly when the sample is longer than i)
 * A: DEVICE float[Hq][pcl_max][pcl_max], C: DEVICE int32[pcl_max]; the caller zeroes both before the first batch.
 *
 * dam_capture_average writes, for every (sequence b, head h) of `shape` (the inputs the masks are for), the
 * averaged map A[h][i][j] / ((float)C[i] + eps) restricted to L_b x L_b (IEEE single division, zero above the
 * diagonal) into P_out, in the layout dam_build_masks_from_scores reads; that call then applies the rule.
 * Both enqueue on `stream`; errors: INVALID_ARGUMENT (null / misaligned pointers, pcl_max < 1, eps <= 0), CUDA.
 */
dam_status_t dam_capture_accumulate(const float* P, const dam_shape_t* shape, int32_t pcl_max, float* A,
                                    int32_t* C, void* stream);
dam_status_t dam_capture_average(const float* A, const int32_t* C, int32_t pcl_max, float eps,
                                 const dam_shape_t* shape, float* P_out, void* stream);

/*
 * Chunked prefill: dam_sparse_attention restricted, per sequence b, to the query rows
 * [row_ranges[2b], row_ranges[2b+1]) (indices inside the sequence). The blob is the one built for the full
 * lengths (stage 1 reads only the first L_b rows of Q and K, so it can be built as soon as the window has been
 * computed); K and V must hold the keys 0 .. end-1 of every sequence, and the rows from `end` up to the next
 * multiple of 128 (as far as the packed buffers reach) must hold finite values: they share a 128-key tile with
 * the last keys, take probability zero, and zero times a NaN or an infinity would still reach the output;
 * rows outside the ranges of O and LSE are neither read nor written. The paper has no counterpart (its Sec. 4.3 extends the mask to "longer sequences"
 * without saying how they arrive); the arithmetic per row is exactly that of dam_sparse_attention.
 * Work is dealt in pairs of 128-row query blocks, so every begin must be a multiple of 256 and every end a
 * multiple of 256 or the sequence length (INVALID_ARGUMENT otherwise); an empty range skips the sequence.
 *   row_ranges_host : HOST, int32[2 * num_seqs] (validated);  row_ranges_dev : DEVICE, the same values.
 * Everything else as dam_sparse_attention.
 */
dam_status_t dam_sparse_attention_rows(const void* Q, const void* K, const void* V, const void* mask,
                                       const dam_shape_t* shape, int32_t causal, int32_t gqa_group,
                                       float softmax_scale, void* O, float* lse,
                                       const int32_t* row_ranges_host, const int32_t* row_ranges_dev,
                                       void* scratch, size_t scratch_bytes, void* stream);

/*
 * Generation-time attention under the stored patterns (Sec. 4.3, Case 2, applied to one new token per
 * sequence; the paper's efficiency table times generation). For every sequence b the query at position
 * i = positions[b] attends, among the keys 0..i of the KV cache, to the keys row i of the extended mask
 * keeps: for i < L_b the row of the true mask; for i >= L_b the matched columns c (V[c] = 1) and the key
 * i - r of every matched diagonal r (D[r] = 1). Only the pattern bits of the blob are read (no tile list), so
 * i may exceed the length the blob was built for. Keys with no active entry: O = 0, LSE = -inf.
 *   q, O : DEVICE, [num_seqs, num_q_heads, head_dim] contiguous, dtype of `shape`. 16-byte aligned.
 *   K, V : DEVICE, the KV cache: sequence b owns rows cu_seqlens[b] .. cu_seqlens[b+1] - 1 (its capacity) of
 *          the packed layout `shape` describes (K / V strides used; Q / O strides ignored); rows 0..i valid.
 *   mask : DEVICE, a blob built for the same number of sequences and query heads (any lengths).
 *   positions_dev : DEVICE, int32[num_seqs], 0 <= positions[b] < capacity of b (checked on the device:
 *          a violation gives O = 0 for that sequence and INVALID_ARGUMENT in the status word of `scratch`).
 *   lse  : DEVICE, float[num_seqs, num_q_heads].   scratch : DEVICE, >= 256 bytes, 256-byte aligned.
 * head_dim 64 or 128 (UNSUPPORTED otherwise). Errors otherwise as dam_sparse_attention.
 */
dam_status_t dam_decode_attention(const void* q, const void* K, const void* V, const void* mask,
                                  const dam_shape_t* shape, const int32_t* positions_dev, int32_t gqa_group,
                                  float softmax_scale, void* O, float* lse, void* scratch,
                                  size_t scratch_bytes, void* stream);

/*
 * Counts taken from a mask blob (DEVICE): out[0] = listed tiles (what the attention kernel executes),
 * out[1] = of those, fully active ones, out[2] = total causal tiles of the shape (for densities),
 * out[3] = bytes of the blob in use (the tile lists have a fixed place per row, sized by the row's upper
 * bound, so this follows from the shapes; out[0] says how many entries are real), out[4] = 128 x 128 tiles of the masks themselves that hold an
 * active cell (equals out[0] unless gathered-column tiles are listed). `out` is HOST memory
 * (5 x uint64). Synchronises `stream` before the header is read.
 * active_elems_dev: DEVICE uint64[num_seqs][num_q_heads], 8-byte aligned, or NULL. When given, a kernel is
 * enqueued on `stream` (not synchronised) that writes, for every (sequence, head), the number of active cells
 * of its S x S mask: the true mask inside the window plus, for every row below it, the matched columns and the
 * matched diagonals with a cell that is both counted once (Sec. 4.3, Case 2; the paper's O(s L) work figure in
 * Sec. 5.3 is this count times 4 d). UNSUPPORTED for a blob made by dam_mask_all_ones.
 * The paper reports no tile counts; they feed the density and active-FLOP figures of the benchmark.
 */
dam_status_t dam_mask_stats(const void* mask, const dam_shape_t* shape, uint64_t* out,
                            uint64_t* active_elems_dev, void* stream);

/*
 * Test hook: expands rows [row_begin, row_begin + nrows) of (seq, head) of the S x S mask exactly as
 * the attention kernels see it (tile list -> tile kind -> per-row 128-bit words, then the causal
 * and sequence-end limits when causal != 0) into out_bits (DEVICE, uint32
 * [nrows][ceil(S / 128) * 4], bit j % 32 of word j / 32 = key j). Lets a test compare the blob with
 * the paper's Case 1 / Case 2 definition (Sec. 4.3) cell by cell.
 */
dam_status_t dam_mask_expand_rows(const void* mask, const dam_shape_t* shape, int32_t seq,
                                  int32_t head, int32_t row_begin, int32_t nrows, int32_t causal,
                                  uint32_t* out_bits, void* stream);

/*
 * Reads the status word at the start of a mask blob or of an attention scratch buffer (DEVICE).
 * Synchronises `stream`, then returns DAM_OK or the recorded device-side status.
 */
dam_status_t dam_poll_status(const void* mask_or_scratch, void* stream);

/*
 * Self-test of the bounded waits the kernels use (every wait on an mbarrier gives up after a time limit,
 * records DAM_ERR_DEVICE_TIMEOUT in the status word and lets the kernel return; nothing spins forever).
 * Launches one tiny kernel that waits, for at most limit_us microseconds (1 .. 1000000), on a barrier
 * nothing arrives on. Afterwards dam_poll_status(scratch, stream) returns DAM_ERR_DEVICE_TIMEOUT and the
 * device stays usable. scratch: DEVICE, >= 256 bytes, 256-byte aligned; bytes 8..15 receive the time waited
 * in nanoseconds. The paper has no counterpart; this exists so that the failure path can be exercised
 * without faulting or hanging a GPU.
 */
dam_status_t dam_selftest_bounded_wait(void* scratch, size_t scratch_bytes, uint32_t limit_us, void* stream);

/*
 * Self-test of the per-device bookkeeping (the paper has no counterpart). The library keeps, per device
 * ordinal, the device's properties and which one-off set-up steps (the shared-memory opt-in of the tensor-core
 * kernels) have run there, in a table guarded by a mutex, so that one process may drive several GPUs from several
 * threads. This call runs the same table code on a private table with a fake device query, for the `n` ordinals
 * given (HOST int32[n]): sm_counts[i] (HOST) receives 100 + ordinal (-1 for an ordinal outside 0..63, and the call
 * then returns INVALID_ARGUMENT), counters[0] (HOST int32[2]) the number of queries made (one per distinct valid
 * ordinal), counters[1] the number of set-up steps run (likewise). No device is touched.
 */
dam_status_t dam_selftest_device_table(const int32_t* ordinals, int32_t n, int32_t* sm_counts, int32_t* counters);

/*
 * Both stages from HOST buffers (pinned recommended, layouts from `shape` with dense strides): copies
 * Q, K, V into the device workspace, runs dam_build_masks and the attention, and copies O and LSE back to
 * HOST. The work is pipelined over chunks of whole query-block pairs in token order: the pattern-capture
 * windows go up first and the masks are built from them; the attention of a chunk (causal: it needs the keys
 * up to the chunk's end only) runs under the upload of the next chunk, and its rows of O and LSE are copied
 * back under both, on two internal streams besides `stream`. All three are synchronised before returning, so
 * the host buffers are complete (and reusable) on return; results are identical to the two device calls.
 * Calls of this entry point are serialised inside the library (one at a time per process).
 * workspace: DEVICE, >= *workspace_bytes as returned when called with workspace == NULL (in that case
 * only the size is computed). The end-to-end figure of the benchmark is measured through this call.
 */
dam_status_t dam_prefill_host(const void* Q_host, const void* K_host, const void* V_host,
                              const dam_shape_t* shape, const dam_rule_t* rule, int32_t causal,
                              void* O_host, float* lse_host, void* workspace,
                              size_t* workspace_bytes, void* stream);

/*
 * Stage 1 for callers that cannot allocate device memory (the paper has no counterpart: this is a
 * packaging variant of dam_build_masks, not a step of the method).  A serving process that gave the
 * whole GPU to its own memory pool, or a loop that must never call cudaMalloc, has no scratch buffer
 * to pass; this call uses a fixed scratch array inside the library instead and allocates nothing
 * (no cudaMalloc, cudaFree or allocating library routine on any path).
 *   - Arguments, layouts, outputs and errors are those of dam_build_masks without `scratch`,
 *     `scratch_bytes` and `scores_dump`; the mask blob written is identical to dam_build_masks'.
 *   - The built-in scratch holds dam_static_scratch_bytes() bytes (8 MiB, enough for 131072 tokens x
 *     32 heads at PCL 4096).  A shape whose build scratch (dam_mask_sizes) is larger is rejected
 *     with DAM_ERR_BUFFER_TOO_SMALL before anything is enqueued.
 *   - Every GPU that loads the library keeps that array until the process exits.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array.  Each call clears the counters it needs, so the
 *     previous call's contents are harmless, but two calls whose GPU work overlaps (different
 *     streams, or threads) race on it: serialise them, or use dam_build_masks with own buffers.
 */
dam_status_t dam_build_masks_static(const void* Q, const void* K, const dam_shape_t* shape,
                                    const dam_rule_t* rule, void* mask, size_t mask_capacity,
                                    void* stream);

/* Size in bytes of the scratch array behind dam_build_masks_static. Host only. */
size_t dam_static_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* DAM_H_ */
