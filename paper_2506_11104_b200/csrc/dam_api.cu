// Host side of the C ABI declared in include/dam.h: argument validation, buffer layout, the
// single-compare form of the threshold, and kernel dispatch.  No device memory is allocated here.
#include <math.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "dam_internal.cuh"

namespace {

struct Layout {
  DamHeader hdr;
  size_t mask_bytes;
  size_t build_scratch_bytes;
  size_t attn_scratch_bytes;
  uint64_t off_cnt, off_cnt_end, off_rowcnt, off_hist, off_cursor, off_items;
  int max_L, max_W, max_nL, max_nq;
  uint64_t score_elems;
};

dam_status_t check_shape(const dam_shape_t* s) {
  if (!s || s->struct_size != sizeof(dam_shape_t)) return DAM_ERR_INVALID_ARGUMENT;
  if (s->num_seqs < 1 || !s->cu_seqlens_host || !s->cu_seqlens_dev) return DAM_ERR_INVALID_ARGUMENT;
  if (s->cu_seqlens_host[0] != 0) return DAM_ERR_INVALID_ARGUMENT;
  for (int b = 0; b < s->num_seqs; ++b) {
    int len = s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b];
    if (len < 0 || len > s->max_seqlen) return DAM_ERR_INVALID_ARGUMENT;
  }
  if (s->cu_seqlens_host[s->num_seqs] != s->total_tokens) return DAM_ERR_INVALID_ARGUMENT;
  if (s->num_q_heads < 1 || s->num_kv_heads < 1 || s->num_q_heads % s->num_kv_heads) return DAM_ERR_INVALID_ARGUMENT;
  if (s->dtype != DAM_BF16 && s->dtype != DAM_F32) return DAM_ERR_INVALID_ARGUMENT;
  if (s->head_dim < 8 || s->head_dim % 8) return DAM_ERR_INVALID_ARGUMENT;
  if (s->head_dim > 256) return DAM_ERR_UNSUPPORTED;
  const int64_t st[8] = {s->q_stride_tok, s->q_stride_head, s->k_stride_tok, s->k_stride_head,
                         s->v_stride_tok, s->v_stride_head, s->o_stride_tok, s->o_stride_head};
  const int64_t vec = s->dtype == DAM_BF16 ? 8 : 4;   // 16-byte vectors
  for (int i = 0; i < 8; ++i)
    if (st[i] < s->head_dim || st[i] % vec) return DAM_ERR_INVALID_ARGUMENT;
  return DAM_OK;
}

dam_status_t check_rule(const dam_rule_t* r) {
  if (!r || r->struct_size != sizeof(dam_rule_t)) return DAM_ERR_INVALID_ARGUMENT;
  if (r->pcl_max < 1) return DAM_ERR_INVALID_ARGUMENT;
  if (!(r->tau > 0.f) || !(r->eps > 0.f) || !(r->mu == r->mu)) return DAM_ERR_INVALID_ARGUMENT;
  if (r->min_support < 1 || (r->flags & ~DAM_RULE_GATHER_COLUMNS) != 0 || r->softmax_scale < 0.f)
    return DAM_ERR_INVALID_ARGUMENT;
  if (r->transform < DAM_TRANSFORM_BOXCOX || r->transform > DAM_TRANSFORM_SUM) return DAM_ERR_INVALID_ARGUMENT;
  if (!(r->lambda == r->lambda) || fabsf(r->lambda) > 64.f) return DAM_ERR_INVALID_ARGUMENT;
  return DAM_OK;
}

bool sm100_shape(const dam_shape_t* s) { return s->dtype == DAM_BF16 && (s->head_dim == 128 || s->head_dim == 64); }

// Gathered-column tiles: asked for by the rule, tensor-core shape, window small enough for the gather kernel.
bool gather_enabled(const dam_shape_t* s, const dam_rule_t* r) {
  return r && (r->flags & DAM_RULE_GATHER_COLUMNS) && sm100_shape(s) && r->pcl_max <= 32768;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Layout of the blob and of the scratch buffers, from the host copy of cu_seqlens.
// pcl_max == 0 selects the all-ones blob (no window sections).
void compute_layout(const dam_shape_t* s, int pcl_max, int all_ones_causal, int gather, Layout* out) {
  Layout& y = *out;
  memset(&y, 0, sizeof(y));
  const int Hq = s->num_q_heads;
  uint64_t dv = 0, tr = 0, cnt = 0, cap = 0, causal_tiles = 0, po = 0, gath = 0;
  int total_qb = 0, total_pairs = 0;
  for (int b = 0; b < s->num_seqs; ++b) {
    int S = s->cu_seqlens_host[b + 1] - s->cu_seqlens_host[b];
    int L = S < pcl_max ? S : pcl_max;
    int W = L > 0 ? dam_words(L) : 0;
    int nL = (L + DAM_TILE - 1) / DAM_TILE;
    int nq = (S + DAM_TILE - 1) / DAM_TILE;
    dv += (uint64_t)Hq * 3 * W;
    tr += (uint64_t)Hq * L * W;
    po += (uint64_t)Hq * L * L;
    cnt += (uint64_t)Hq * dam_cnt_stride(L, W, nL);
    gath += (uint64_t)Hq * nL;
    causal_tiles += (uint64_t)Hq * nq * (nq + 1) / 2;
    if (pcl_max > 0) {
      for (int qb = 0; qb < nq; ++qb) cap += (uint64_t)Hq * dam_row_tile_bound(qb, nL, L, gather);
    } else {
      cap += (uint64_t)Hq * (all_ones_causal ? (uint64_t)nq * (nq + 1) / 2 : (uint64_t)nq * nq);
    }
    total_qb += nq;
    total_pairs += (nq + 1) / 2;
    if (L > y.max_L) y.max_L = L;
    if (W > y.max_W) y.max_W = W;
    if (nL > y.max_nL) y.max_nL = nL;
    if (nq > y.max_nq) y.max_nq = nq;
  }
  DamHeader& h = y.hdr;
  h.magic = DAM_MAGIC;
  h.status = 0;
  h.version = 1;
  h.flags = pcl_max > 0 ? (DAM_FLAG_CAUSAL_LIST | (gather ? DAM_FLAG_GATHER : 0u))
                        : (DAM_FLAG_ALL_ONES | (all_ones_causal ? DAM_FLAG_CAUSAL_LIST : 0u));
  h.num_seqs = s->num_seqs;
  h.num_q_heads = Hq;
  h.total_qblocks = total_qb;
  h.rows = Hq * total_qb;
  h.total_pairs = total_pairs;
  h.prows = Hq * total_pairs;
  h.tile_capacity = (uint32_t)(cap > 0xFFFFFFF0ull ? 0xFFFFFFF0ull : cap);
  h.pcl_max = (uint32_t)pcl_max;
  h.off_seq = sizeof(DamHeader);
  h.off_qbseq = dam_align(h.off_seq + (uint64_t)s->num_seqs * sizeof(DamSeq), 256);
  h.off_pairtab = dam_align(h.off_qbseq + 4ull * total_qb, 256);
  h.off_dv = dam_align(h.off_pairtab + 4ull * total_pairs, 256);
  h.off_true = dam_align(h.off_dv + 4ull * dv, 256);
  h.off_tile_ptr = dam_align(h.off_true + 4ull * tr, 256);
  h.off_work = dam_align(h.off_tile_ptr + 4ull * (h.rows + 1), 256);
  h.off_tiles = dam_align(h.off_work + (uint64_t)sizeof(DamItem) * h.prows, 256);
  h.causal_tiles = causal_tiles;
  y.mask_bytes = dam_align(h.off_tiles + 4ull * cap, 256);
  // build scratch: [0,256) status block and work counter | counts | row counts | hist | cursor | unordered items
  y.off_cnt = 256;
  y.off_cnt_end = dam_align(y.off_cnt + 4ull * cnt, 256);
  y.off_rowcnt = y.off_cnt_end;
  y.off_hist = dam_align(y.off_rowcnt + 4ull * h.rows, 256);
  y.off_cursor = y.off_hist + 4ull * DAM_HIST;
  y.off_items = dam_align(y.off_cursor + 4ull * DAM_HIST, 256);          // work items before they are ordered
  y.build_scratch_bytes = dam_align(y.off_items + (uint64_t)sizeof(DamItem) * h.prows, 256);
  // attention scratch: 256-byte status block, then (gathered columns only) one K tile and one V tile of
  // 128 keys per gathered-column tile
  h.gath_tiles = (pcl_max > 0 && gather) ? gath : 0;
  y.attn_scratch_bytes = 256 + h.gath_tiles * 2ull * DAM_TILE * s->head_dim * 2ull;
  h.attn_scratch_bytes = y.attn_scratch_bytes;
  y.score_elems = po;
}

// The threshold chain of the true mask (Sec. 4.2.2 - 4.2.3 with lambda = 0.5), each step one IEEE
// single-precision operation:  x = max(p, eps); b = (sqrt(x) - 1) * 2; a = b - (sqrt(eps) - 1) * 2;
// active = a >= tau.  Every step is monotone in p, so the active set is {p >= p*}; p* is found by
// bisection over the float bit patterns in [0, 1] and the kernels use the single compare.
bool chain_active(float p, float tau, float eps) {
  volatile float x = p > eps ? p : eps;
  volatile float r = sqrtf(x);
  volatile float b = (r - 1.0f) * 2.0f;
  volatile float se = sqrtf(eps);
  volatile float bmin = (se - 1.0f) * 2.0f;
  volatile float a = b - bmin;
  return a >= tau;
}

// Every other amplification (Appendix B), decided in double precision on the fp32 map value.
double amplify_f64(double X, int transform, double lam) {
  switch (transform) {
    case DAM_TRANSFORM_BOXCOX: return lam == 0.0 ? log(X) : (pow(X, lam) - 1.0) / lam;
    case DAM_TRANSFORM_LOG: return log(X);
    case DAM_TRANSFORM_SQRT: return sqrt(X);
    case DAM_TRANSFORM_ARCSINH: return asinh(X);
    case DAM_TRANSFORM_YEO_JOHNSON: return lam == 0.0 ? log(X + 1.0) : (pow(X + 1.0, lam) - 1.0) / lam;
    default: return X;
  }
}

struct Rule64 { int transform; double tau, eps, lam; bool chain; float ftau, feps; };

bool rule_active(float p, const Rule64& r) {
  if (r.chain) return chain_active(p, r.ftau, r.feps);
  const double X = (double)p > r.eps ? (double)p : r.eps;
  return amplify_f64(X, r.transform, r.lam) - amplify_f64(r.eps, r.transform, r.lam) >= r.tau;
}

float find_pstar(const dam_rule_t* rule) {
  Rule64 r;
  r.transform = rule->transform; r.tau = (double)rule->tau; r.eps = (double)rule->eps; r.lam = (double)rule->lambda;
  r.chain = rule->transform == DAM_TRANSFORM_BOXCOX && rule->lambda == 0.5f;
  r.ftau = rule->tau; r.feps = rule->eps;
  if (!rule_active(1.0f, r)) {
    // no probability reaches tau; larger (non-softmax) inputs may: search up to the largest float
    uint32_t lo = 0x3F800000u, hi = 0x7F7FFFFFu;
    float fh; memcpy(&fh, &hi, 4);
    if (!rule_active(fh, r)) return INFINITY;
    while (hi - lo > 1) {
      uint32_t mid = lo + (hi - lo) / 2; float fm; memcpy(&fm, &mid, 4);
      if (rule_active(fm, r)) hi = mid; else lo = mid;
    }
    memcpy(&fh, &hi, 4);
    return fh;
  }
  uint32_t lo = 0u, hi = 0x3F800000u;     // the rule is inactive at 0 because tau > 0
  while (hi - lo > 1) {
    uint32_t mid = lo + (hi - lo) / 2; float fm; memcpy(&fm, &mid, 4);
    if (rule_active(fm, r)) hi = mid; else lo = mid;
  }
  float f; memcpy(&f, &hi, 4);
  return f;
}

dam_status_t fill_ctx(const dam_shape_t* s, const dam_rule_t* r, void* mask, size_t cap, void* scratch,
                      size_t scratch_bytes, Layout* y, DamBuildCtx* c) {
  dam_status_t st;
  if ((st = check_shape(s)) != DAM_OK) return st;
  if ((st = check_rule(r)) != DAM_OK) return st;
  if (!mask || !scratch || !aligned(mask, 256) || !aligned(scratch, 256)) return DAM_ERR_INVALID_ARGUMENT;
  const int gather = gather_enabled(s, r);
  compute_layout(s, r->pcl_max, 1, gather, y);
  if (cap < y->mask_bytes || scratch_bytes < y->build_scratch_bytes) return DAM_ERR_BUFFER_TOO_SMALL;
  c->blob = reinterpret_cast<unsigned char*>(mask);
  c->scratch = reinterpret_cast<unsigned char*>(scratch);
  c->num_seqs = s->num_seqs; c->Hq = s->num_q_heads; c->Hkv = s->num_kv_heads; c->d = s->head_dim; c->dtype = s->dtype;
  c->total_qblocks = y->hdr.total_qblocks; c->rows = y->hdr.rows; c->prows = y->hdr.prows;
  c->max_L = y->max_L; c->max_W = y->max_W; c->max_nL = y->max_nL; c->max_nq = y->max_nq;
  c->per_map = (r->transform == DAM_TRANSFORM_ZSCORE || r->transform == DAM_TRANSFORM_MINMAX) ? r->transform : 0;
  c->tau = r->tau; c->eps = r->eps;
  c->pstar = c->per_map ? INFINITY : find_pstar(r);
  c->mu = r->mu; c->min_support = r->min_support;
  c->scale = r->softmax_scale > 0.f ? r->softmax_scale : 1.0f / sqrtf((float)s->head_dim);
  c->off_cnt = y->off_cnt; c->off_cnt_end = y->off_cnt_end; c->off_rowcnt = y->off_rowcnt; c->off_items = y->off_items;
  c->off_hist = y->off_hist; c->off_cursor = y->off_cursor;
  c->gather = gather;
  c->off_true = y->hdr.off_true; c->true_bytes = y->hdr.off_tile_ptr - y->hdr.off_true;
  return DAM_OK;
}

std::mutex g_device_mutex;

cudaError_t query_device(int device, DamDeviceInfo* out) {
  cudaError_t e;
  if ((e = cudaDeviceGetAttribute(&out->cc_major, cudaDevAttrComputeCapabilityMajor, device)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&out->sm_count, cudaDevAttrMultiProcessorCount, device)) != cudaSuccess) return e;
  return cudaDeviceGetAttribute(&out->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
}

}  // namespace

cudaError_t DamDeviceTable::info(int device, dam_device_query_fn query, DamDeviceInfo* out) {
  if (device < 0 || device >= kMaxDevices || !query || !out) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  Slot& s = slots_[device];
  if (!s.filled) {
    DamDeviceInfo di = {};
    const cudaError_t e = query(device, &di);
    if (e != cudaSuccess) return e;                 // nothing is remembered about a failed query
    s.info = di;
    s.filled = true;
  }
  *out = s.info;
  return cudaSuccess;
}

cudaError_t DamDeviceTable::once(int device, int key, dam_device_setup_fn fn) {
  if (device < 0 || device >= kMaxDevices || key < 0 || key >= kMaxSetups || !fn) return cudaErrorInvalidValue;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  Slot& s = slots_[device];
  if (s.done[key]) return cudaSuccess;
  const cudaError_t e = fn();
  if (e == cudaSuccess) s.done[key] = true;
  return e;
}

DamDeviceTable& dam_device_table() {
  static DamDeviceTable table;
  return table;
}

cudaError_t dam_current_device(int* device, DamDeviceInfo* info) {
  cudaError_t e = cudaGetDevice(device);
  if (e != cudaSuccess) return e;
  return dam_device_table().info(*device, query_device, info);
}

extern "C" {

int32_t dam_version(void) { return 1001; }

const char* dam_status_string(dam_status_t s) {
  switch (s) {
    case DAM_OK: return "ok";
    case DAM_ERR_INVALID_ARGUMENT: return "invalid argument";
    case DAM_ERR_UNSUPPORTED: return "unsupported";
    case DAM_ERR_BUFFER_TOO_SMALL: return "buffer too small";
    case DAM_ERR_CUDA: return "CUDA error";
    case DAM_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case DAM_ERR_INTERNAL: return "internal error";
  }
  return "unknown status";
}

dam_status_t dam_mask_sizes(const dam_shape_t* shape, const dam_rule_t* rule, int32_t causal, size_t* mask_bytes,
                            size_t* build_scratch_bytes, size_t* attn_scratch_bytes) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (rule && (st = check_rule(rule)) != DAM_OK) return st;
  Layout y;
  compute_layout(shape, rule ? rule->pcl_max : 0, causal != 0,
                 gather_enabled(shape, rule), &y);
  if (mask_bytes) *mask_bytes = y.mask_bytes;
  if (build_scratch_bytes) *build_scratch_bytes = rule ? y.build_scratch_bytes : 0;
  if (attn_scratch_bytes) *attn_scratch_bytes = y.attn_scratch_bytes;
  return DAM_OK;
}

dam_status_t dam_build_masks(const void* Q, const void* K, const dam_shape_t* shape, const dam_rule_t* rule,
                             void* mask, size_t mask_capacity, void* scratch, size_t scratch_bytes,
                             float* scores_dump, void* stream) {
  Layout y; DamBuildCtx c;
  dam_status_t st = fill_ctx(shape, rule, mask, mask_capacity, scratch, scratch_bytes, &y, &c);
  if (st != DAM_OK) return st;
  if (!Q || !K || !aligned(Q, 16) || !aligned(K, 16) || (scores_dump && !aligned(scores_dump, 16)))
    return DAM_ERR_INVALID_ARGUMENT;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  // thresholds from a map's own statistics need the finished map: with a dump buffer the map is written there first
  // and thresholded in a second pass; without one the caller has to go through dam_build_masks_from_scores
  if (c.per_map && !scores_dump) return DAM_ERR_UNSUPPORTED;
  if (dam_launch_rule_prepare(c, cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (dam_launch_init_blob(shape, rule->pcl_max, y.hdr.flags, mask, y.hdr, cs) != cudaSuccess)
    return DAM_ERR_CUDA;
  cudaError_t e = cudaErrorNotSupported;
  if (sm100_shape(shape)) e = dam_launch_scores_sm100(Q, K, shape, c, scores_dump, cs);
  if (e == cudaErrorNotSupported) e = dam_launch_scores_ref(Q, K, shape, c, scores_dump, cs);
  if (e != cudaSuccess) return DAM_ERR_CUDA;
  if (c.per_map && dam_launch_bits_from_scores(scores_dump, c, cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (dam_launch_rule(c, cs) != cudaSuccess) return DAM_ERR_CUDA;
  return DAM_OK;
}

dam_status_t dam_build_masks_from_scores(const float* P, const dam_shape_t* shape, const dam_rule_t* rule,
                                         void* mask, size_t mask_capacity, void* scratch, size_t scratch_bytes,
                                         void* stream) {
  Layout y; DamBuildCtx c;
  dam_status_t st = fill_ctx(shape, rule, mask, mask_capacity, scratch, scratch_bytes, &y, &c);
  if (st != DAM_OK) return st;
  if (!P || !aligned(P, 4)) return DAM_ERR_INVALID_ARGUMENT;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  if (dam_launch_rule_prepare(c, cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (dam_launch_init_blob(shape, rule->pcl_max, y.hdr.flags, mask, y.hdr, cs) != cudaSuccess)
    return DAM_ERR_CUDA;
  if (dam_launch_bits_from_scores(P, c, cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (dam_launch_rule(c, cs) != cudaSuccess) return DAM_ERR_CUDA;
  return DAM_OK;
}

dam_status_t dam_capture_accumulate(const float* P, const dam_shape_t* shape, int32_t pcl_max, float* A, int32_t* C,
                                    void* stream) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (!P || !A || !C || pcl_max < 1 || !aligned(P, 4) || !aligned(A, 4) || !aligned(C, 4)) return DAM_ERR_INVALID_ARGUMENT;
  return dam_launch_capture_accumulate(P, shape, pcl_max, A, C, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
             ? DAM_OK : DAM_ERR_CUDA;
}

dam_status_t dam_capture_average(const float* A, const int32_t* C, int32_t pcl_max, float eps,
                                 const dam_shape_t* shape, float* P_out, void* stream) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (!A || !C || !P_out || pcl_max < 1 || !(eps > 0.f) || !aligned(P_out, 4) || !aligned(A, 4) || !aligned(C, 4))
    return DAM_ERR_INVALID_ARGUMENT;
  return dam_launch_capture_average(A, C, pcl_max, eps, shape, P_out, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
             ? DAM_OK : DAM_ERR_CUDA;
}

dam_status_t dam_mask_all_ones(const dam_shape_t* shape, int32_t causal, void* mask, size_t mask_capacity,
                               void* stream) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (!mask || !aligned(mask, 256)) return DAM_ERR_INVALID_ARGUMENT;
  Layout y;
  compute_layout(shape, 0, causal != 0, 0, &y);
  if (mask_capacity < y.mask_bytes) return DAM_ERR_BUFFER_TOO_SMALL;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  if (dam_launch_init_blob(shape, 0, y.hdr.flags, mask, y.hdr, cs) != cudaSuccess)
    return DAM_ERR_CUDA;
  if (dam_launch_all_ones(shape, causal != 0, mask, cs) != cudaSuccess) return DAM_ERR_CUDA;
  return DAM_OK;
}

static dam_status_t sparse_attention_impl(const void* Q, const void* K, const void* V, const void* mask,
                                          const dam_shape_t* shape, int32_t causal, int32_t gqa_group,
                                          float softmax_scale, void* O, float* lse, const int32_t* ranges_host,
                                          const int32_t* ranges_dev, void* scratch, size_t scratch_bytes,
                                          void* stream, bool continuation = false) {
  // continuation: a further row range of the same layer against the same scratch buffer: the status word is
  // kept, and the gathered-column tiles the first call built are used again
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (!Q || !K || !V || !mask || !O || !lse || !scratch) return DAM_ERR_INVALID_ARGUMENT;
  if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(lse, 4) ||
      !aligned(mask, 256) || !aligned(scratch, 256))
    return DAM_ERR_INVALID_ARGUMENT;
  if (gqa_group != shape->num_q_heads / shape->num_kv_heads || softmax_scale < 0.f) return DAM_ERR_INVALID_ARGUMENT;
  if ((ranges_host == nullptr) != (ranges_dev == nullptr)) return DAM_ERR_INVALID_ARGUMENT;
  if (ranges_host) {
    if (!aligned(ranges_dev, 4)) return DAM_ERR_INVALID_ARGUMENT;
    for (int b = 0; b < shape->num_seqs; ++b) {
      const int S = shape->cu_seqlens_host[b + 1] - shape->cu_seqlens_host[b];
      const int r0 = ranges_host[2 * b], r1 = ranges_host[2 * b + 1];
      // whole pairs of query blocks: begin on a multiple of 256, end on a multiple of 256 or the sequence end
      if (r0 < 0 || r1 < r0 || r1 > S || r0 % (2 * DAM_TILE) || (r1 % (2 * DAM_TILE) && r1 != S))
        return DAM_ERR_INVALID_ARGUMENT;
    }
  }
  if (scratch_bytes < 256) return DAM_ERR_BUFFER_TOO_SMALL;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)shape->head_dim);
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  // status word and work counter start at zero (a continuation clears the work counter only)
  if (cudaMemsetAsync(reinterpret_cast<unsigned char*>(scratch) + (continuation ? 8 : 0), 0, continuation ? 248 : 256, cs) !=
      cudaSuccess)
    return DAM_ERR_CUDA;
  cudaError_t e = cudaErrorNotSupported;
  if (sm100_shape(shape))
    e = dam_launch_attn_sm100(Q, K, V, mask, shape, causal != 0, scale, O, lse, scratch, scratch_bytes, ranges_dev,
                              !continuation, cs);
  if (e == cudaErrorNotSupported)
    e = dam_launch_attn_ref(Q, K, V, mask, shape, causal != 0, scale, O, lse, scratch, ranges_dev, cs);
  return e == cudaSuccess ? DAM_OK : DAM_ERR_CUDA;
}

dam_status_t dam_sparse_attention(const void* Q, const void* K, const void* V, const void* mask,
                                  const dam_shape_t* shape, int32_t causal, int32_t gqa_group, float softmax_scale,
                                  void* O, float* lse, void* scratch, size_t scratch_bytes, void* stream) {
  return sparse_attention_impl(Q, K, V, mask, shape, causal, gqa_group, softmax_scale, O, lse, nullptr, nullptr,
                               scratch, scratch_bytes, stream);
}

dam_status_t dam_sparse_attention_rows(const void* Q, const void* K, const void* V, const void* mask,
                                       const dam_shape_t* shape, int32_t causal, int32_t gqa_group,
                                       float softmax_scale, void* O, float* lse, const int32_t* row_ranges_host,
                                       const int32_t* row_ranges_dev, void* scratch, size_t scratch_bytes,
                                       void* stream) {
  if (!row_ranges_host || !row_ranges_dev) return DAM_ERR_INVALID_ARGUMENT;
  return sparse_attention_impl(Q, K, V, mask, shape, causal, gqa_group, softmax_scale, O, lse, row_ranges_host,
                               row_ranges_dev, scratch, scratch_bytes, stream);
}

dam_status_t dam_decode_attention(const void* q, const void* K, const void* V, const void* mask,
                                  const dam_shape_t* shape, const int32_t* positions_dev, int32_t gqa_group,
                                  float softmax_scale, void* O, float* lse, void* scratch, size_t scratch_bytes,
                                  void* stream) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (!q || !K || !V || !mask || !positions_dev || !O || !lse || !scratch) return DAM_ERR_INVALID_ARGUMENT;
  if (!aligned(q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(O, 16) || !aligned(lse, 4) ||
      !aligned(positions_dev, 4) || !aligned(mask, 256) || !aligned(scratch, 256))
    return DAM_ERR_INVALID_ARGUMENT;
  if (gqa_group != shape->num_q_heads / shape->num_kv_heads || softmax_scale < 0.f) return DAM_ERR_INVALID_ARGUMENT;
  if (shape->head_dim != 64 && shape->head_dim != 128) return DAM_ERR_UNSUPPORTED;
  if (scratch_bytes < 256) return DAM_ERR_BUFFER_TOO_SMALL;
  const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)shape->head_dim);
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(scratch, 0, 256, cs) != cudaSuccess) return DAM_ERR_CUDA;
  cudaError_t e = dam_launch_decode(q, K, V, mask, shape, positions_dev, scale, O, lse, scratch, cs);
  if (e == cudaErrorNotSupported) return DAM_ERR_UNSUPPORTED;
  return e == cudaSuccess ? DAM_OK : DAM_ERR_CUDA;
}

dam_status_t dam_mask_stats(const void* mask, const dam_shape_t* shape, uint64_t* out, uint64_t* active_elems_dev,
                            void* stream) {
  if (!mask || !out || !shape) return DAM_ERR_INVALID_ARGUMENT;
  if (active_elems_dev && !aligned(active_elems_dev, 8)) return DAM_ERR_INVALID_ARGUMENT;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  DamHeader h;
  if (cudaMemcpyAsync(&h, mask, sizeof(h), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (h.magic != DAM_MAGIC) return DAM_ERR_INVALID_ARGUMENT;
  if (active_elems_dev) {
    if (h.flags & DAM_FLAG_ALL_ONES) return DAM_ERR_UNSUPPORTED;      // an all-ones blob has no pattern sections
    if (h.num_seqs != shape->num_seqs || h.num_q_heads != shape->num_q_heads) return DAM_ERR_INVALID_ARGUMENT;
    if (dam_launch_active_elems(mask, h.num_seqs, h.num_q_heads, reinterpret_cast<unsigned long long*>(active_elems_dev),
                                cs) != cudaSuccess)
      return DAM_ERR_CUDA;
  }
  out[0] = h.total_tiles; out[1] = h.full_tiles; out[2] = h.causal_tiles; out[3] = h.bytes_used;
  out[4] = h.mask_tiles;
  return DAM_OK;
}

dam_status_t dam_mask_expand_rows(const void* mask, const dam_shape_t* shape, int32_t seq, int32_t head,
                                  int32_t row_begin, int32_t nrows, int32_t causal, uint32_t* out_bits,
                                  void* stream) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if (!mask || !out_bits || seq < 0 || seq >= shape->num_seqs || head < 0 || head >= shape->num_q_heads ||
      nrows < 0 || row_begin < 0)
    return DAM_ERR_INVALID_ARGUMENT;
  if (nrows == 0) return DAM_OK;
  int S = shape->cu_seqlens_host[seq + 1] - shape->cu_seqlens_host[seq];
  int words = ((S + DAM_TILE - 1) / DAM_TILE) * 4;
  if (words == 0) return DAM_OK;
  cudaError_t e = dam_launch_expand_rows(mask, seq, head, row_begin, nrows, words, causal != 0, out_bits,
                                         reinterpret_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? DAM_OK : DAM_ERR_CUDA;
}

dam_status_t dam_poll_status(const void* mask_or_scratch, void* stream) {
  if (!mask_or_scratch) return DAM_ERR_INVALID_ARGUMENT;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  uint32_t w[2] = {0, 0};
  if (cudaMemcpyAsync(w, mask_or_scratch, sizeof(w), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (cudaStreamSynchronize(cs) != cudaSuccess) return DAM_ERR_CUDA;
  if (w[1] > DAM_ERR_INTERNAL) return DAM_ERR_INTERNAL;
  return static_cast<dam_status_t>(w[1]);
}

dam_status_t dam_selftest_bounded_wait(void* scratch, size_t scratch_bytes, uint32_t limit_us, void* stream) {
  if (!scratch || !aligned(scratch, 256) || limit_us == 0 || limit_us > 1000000u) return DAM_ERR_INVALID_ARGUMENT;
  if (scratch_bytes < 256) return DAM_ERR_BUFFER_TOO_SMALL;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(scratch, 0, 256, cs) != cudaSuccess) return DAM_ERR_CUDA;
  return dam_launch_bounded_wait_selftest(scratch, 1000ull * limit_us, cs) == cudaSuccess ? DAM_OK : DAM_ERR_CUDA;
}

namespace {
int g_fake_queries = 0;
cudaError_t fake_query(int device, DamDeviceInfo* out) {
  ++g_fake_queries;                                  // (called under the table's lock)
  out->cc_major = 10; out->sm_count = 100 + device; out->smem_optin = 1000 * (device + 1);
  return cudaSuccess;
}
int g_fake_setups = 0;
cudaError_t fake_setup() { ++g_fake_setups; return cudaSuccess; }
}  // namespace

dam_status_t dam_selftest_device_table(const int32_t* ordinals, int32_t n, int32_t* sm_counts, int32_t* counters) {
  if (!ordinals || !sm_counts || !counters || n < 0) return DAM_ERR_INVALID_ARGUMENT;
  static std::mutex selftest_mutex;
  std::lock_guard<std::mutex> lock(selftest_mutex);
  DamDeviceTable table;                              // a table of its own: the library's records are not touched
  g_fake_queries = g_fake_setups = 0;
  dam_status_t st = DAM_OK;
  for (int i = 0; i < n; ++i) {
    DamDeviceInfo di = {};
    if (table.info(ordinals[i], fake_query, &di) != cudaSuccess ||
        table.once(ordinals[i], DAM_SETUP_ATTN_SMEM, fake_setup) != cudaSuccess) {
      sm_counts[i] = -1;
      st = DAM_ERR_INVALID_ARGUMENT;
      continue;
    }
    sm_counts[i] = di.sm_count;
  }
  counters[0] = g_fake_queries;
  counters[1] = g_fake_setups;
  return st;
}

// Streams and events of the host-buffer entry point (created on first use, one set per device).
namespace {
constexpr int kMaxChunks = 32;
struct HostPipe {
  bool ready = false;
  cudaStream_t h2d = nullptr, d2h = nullptr;
  cudaEvent_t start = nullptr, window = nullptr, out = nullptr, up[kMaxChunks] = {}, done[kMaxChunks] = {};
};
std::mutex g_pipe_mutex;
HostPipe g_pipes[64];

HostPipe* host_pipe() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPipe& p = g_pipes[dev];
  if (p.ready) return &p;
  bool ok = cudaStreamCreateWithFlags(&p.h2d, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&p.d2h, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.window, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&p.out, cudaEventDisableTiming) == cudaSuccess;
  for (int c = 0; ok && c < kMaxChunks; ++c)
    ok = cudaEventCreateWithFlags(&p.up[c], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&p.done[c], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) return nullptr;
  p.ready = true;
  return &p;
}
}  // namespace

// The copies and the kernels are pipelined over chunks of whole query-block pairs, in token order.  First the
// pattern-capture windows of all sequences go up (rows [0, L) of Q, K, V: all the mask construction and the
// gathered-column tiles read); while the masks are built the first chunk follows.  The attention of chunk c
// (dam_sparse_attention_rows on its row ranges; causal, so it needs the keys up to the chunk's end only) runs as
// soon as the chunk is on the device, under the upload of chunk c + 1, and its rows of O and LSE go back to the
// host on a third stream under both.  Uploads use one PCIe direction and downloads the other.
dam_status_t dam_prefill_host(const void* Qh, const void* Kh, const void* Vh, const dam_shape_t* shape,
                              const dam_rule_t* rule, int32_t causal, void* Oh, float* lse_h, void* workspace,
                              size_t* workspace_bytes, void* stream) {
  dam_status_t st;
  if ((st = check_shape(shape)) != DAM_OK) return st;
  if ((st = check_rule(rule)) != DAM_OK) return st;
  if (!workspace_bytes) return DAM_ERR_INVALID_ARGUMENT;
  const size_t es = shape->dtype == DAM_BF16 ? 2 : 4;
  const int64_t T = shape->total_tokens, Hq = shape->num_q_heads, Hkv = shape->num_kv_heads, d = shape->head_dim;
  const int nb = shape->num_seqs;
  // dense strides only
  if (shape->q_stride_head != d || shape->q_stride_tok != Hq * d || shape->k_stride_head != d ||
      shape->k_stride_tok != Hkv * d || shape->v_stride_head != d || shape->v_stride_tok != Hkv * d ||
      shape->o_stride_head != d || shape->o_stride_tok != Hq * d)
    return DAM_ERR_UNSUPPORTED;
  Layout y;
  compute_layout(shape, rule->pcl_max, 1, gather_enabled(shape, rule), &y);
  const size_t qb = dam_align((size_t)T * Hq * d * es, 256), kb = dam_align((size_t)T * Hkv * d * es, 256);
  const size_t lb = dam_align((size_t)Hq * T * 4, 256);
  const size_t rb = dam_align((size_t)kMaxChunks * 2 * (size_t)(nb > 0 ? nb : 1) * sizeof(int32_t), 256);
  size_t off_q = 0, off_k = off_q + qb, off_v = off_k + kb, off_o = off_v + kb, off_l = off_o + qb;
  size_t off_m = off_l + lb, off_bs = off_m + y.mask_bytes, off_as = off_bs + y.build_scratch_bytes;
  size_t off_r = off_as + dam_align(y.attn_scratch_bytes, 256);
  size_t total = off_r + rb;
  if (!workspace) { *workspace_bytes = total; return DAM_OK; }
  if (*workspace_bytes < total) return DAM_ERR_BUFFER_TOO_SMALL;
  if (!Qh || !Kh || !Vh || !Oh || !lse_h || !aligned(workspace, 256)) return DAM_ERR_INVALID_ARGUMENT;
  cudaStream_t cs = reinterpret_cast<cudaStream_t>(stream);
  unsigned char* w = reinterpret_cast<unsigned char*>(workspace);
  if (T == 0) return cudaStreamSynchronize(cs) == cudaSuccess ? DAM_OK : DAM_ERR_CUDA;

  // ---- chunk plan: pieces of whole query-block pairs of one sequence, grouped in token order
  const int* cu = shape->cu_seqlens_host;
  int64_t chunk_rows = (T / 8 + 255) / 256 * 256;          // eight chunks: more gave nothing on PCIe 5 x16
  if (chunk_rows < 2048) chunk_rows = 2048;
  struct Chunk { int64_t t0, t1; };
  std::vector<Chunk> chunks;
  std::vector<int32_t> ranges;                 // [chunk][2 * seq]
  for (;;) {
    chunks.clear(); ranges.clear();
    for (int b = 0; b < nb; ++b) {
      const int S = cu[b + 1] - cu[b];
      for (int64_t r0 = 0; r0 < S; r0 += chunk_rows) {
        const int64_t r1 = r0 + chunk_rows < S ? r0 + chunk_rows : S;
        const bool fresh = chunks.empty() || (chunks.back().t1 - chunks.back().t0) + (r1 - r0) > chunk_rows;
        if (fresh) {
          chunks.push_back({cu[b] + r0, cu[b] + r0});
          ranges.resize(ranges.size() + 2 * (size_t)nb, 0);
        }
        int32_t* rg = ranges.data() + (chunks.size() - 1) * 2 * (size_t)nb;
        if (rg[2 * b + 1] == 0) rg[2 * b] = (int32_t)r0;
        rg[2 * b + 1] = (int32_t)r1;
        chunks.back().t1 = cu[b] + r1;
      }
    }
    if ((int)chunks.size() <= kMaxChunks) break;
    chunk_rows *= 2;
  }
  const int nc = (int)chunks.size();

  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe* pp = host_pipe();
  if (!pp) return DAM_ERR_CUDA;
  HostPipe& P = *pp;
  const char* Qc = reinterpret_cast<const char*>(Qh);
  const char* Kc = reinterpret_cast<const char*>(Kh);
  const char* Vc = reinterpret_cast<const char*>(Vh);
  const size_t qrow = (size_t)Hq * d * es, krow = (size_t)Hkv * d * es;
  bool ok = true;
  auto up = [&](int64_t a, int64_t e, bool with_qk) {   // tokens [a, e): V always, Q and K unless already up
    if (e <= a || !ok) return;
    if (with_qk)
      ok = cudaMemcpyAsync(w + off_q + a * qrow, Qc + a * qrow, (size_t)(e - a) * qrow, cudaMemcpyHostToDevice, P.h2d) == cudaSuccess &&
           cudaMemcpyAsync(w + off_k + a * krow, Kc + a * krow, (size_t)(e - a) * krow, cudaMemcpyHostToDevice, P.h2d) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(w + off_v + a * krow, Vc + a * krow, (size_t)(e - a) * krow, cudaMemcpyHostToDevice, P.h2d) == cudaSuccess;
  };
  // the workspace may still be in use by earlier work of the caller's stream
  ok = cudaEventRecord(P.start, cs) == cudaSuccess && cudaStreamWaitEvent(P.h2d, P.start, 0) == cudaSuccess &&
       cudaStreamWaitEvent(P.d2h, P.start, 0) == cudaSuccess;
  // A chunk that ends at a sequence end inside a 128-key tile makes that tile's K / V rows reach into tokens that
  // arrive with a later chunk; their probabilities are zero, but a zero times whatever bytes the workspace held
  // (a NaN or an infinity) is not: K and V start out as zeros.
  ok = ok && cudaMemsetAsync(w + off_k, 0, kb, P.h2d) == cudaSuccess && cudaMemsetAsync(w + off_v, 0, kb, P.h2d) == cudaSuccess;
  // windows first, with the row ranges of all chunks
  ok = ok && cudaMemcpyAsync(w + off_r, ranges.data(), ranges.size() * sizeof(int32_t), cudaMemcpyHostToDevice, P.h2d) == cudaSuccess;
  for (int b = 0; b < nb && ok; ++b) {
    const int S = cu[b + 1] - cu[b];
    const int L = S < rule->pcl_max ? S : rule->pcl_max;
    up(cu[b], cu[b] + L, true);
  }
  ok = ok && cudaEventRecord(P.window, P.h2d) == cudaSuccess && cudaStreamWaitEvent(cs, P.window, 0) == cudaSuccess;
  if (!ok) return DAM_ERR_CUDA;
  st = dam_build_masks(w + off_q, w + off_k, shape, rule, w + off_m, y.mask_bytes, w + off_bs, y.build_scratch_bytes,
                       nullptr, stream);
  if (st != DAM_OK) { cudaStreamSynchronize(P.h2d); return st; }
  int b_lo = 0;
  for (int c = 0; c < nc && ok; ++c) {
    const int64_t t0 = chunks[c].t0, t1 = chunks[c].t1;
    // the rest of the chunk: per sequence, what lies below its window
    while (b_lo + 1 < nb && cu[b_lo + 1] <= t0) ++b_lo;
    for (int b = b_lo; b < nb && cu[b] < t1; ++b) {
      const int S = cu[b + 1] - cu[b];
      const int L = S < rule->pcl_max ? S : rule->pcl_max;
      const int64_t a = t0 > cu[b] + L ? t0 : cu[b] + L, e = t1 < cu[b + 1] ? t1 : cu[b + 1];
      up(a, e, true);
    }
    ok = ok && cudaEventRecord(P.up[c], P.h2d) == cudaSuccess && cudaStreamWaitEvent(cs, P.up[c], 0) == cudaSuccess;
    if (!ok) break;
    const int32_t* rg = ranges.data() + (size_t)c * 2 * nb;
    st = sparse_attention_impl(w + off_q, w + off_k, w + off_v, w + off_m, shape, causal,
                               shape->num_q_heads / shape->num_kv_heads, rule->softmax_scale, w + off_o,
                               reinterpret_cast<float*>(w + off_l), rg,
                               reinterpret_cast<const int32_t*>(w + off_r) + (size_t)c * 2 * nb, w + off_as,
                               y.attn_scratch_bytes, stream, c > 0);
    if (st != DAM_OK) break;
    ok = cudaEventRecord(P.done[c], cs) == cudaSuccess && cudaStreamWaitEvent(P.d2h, P.done[c], 0) == cudaSuccess &&
         cudaMemcpyAsync(reinterpret_cast<char*>(Oh) + t0 * qrow, w + off_o + t0 * qrow, (size_t)(t1 - t0) * qrow,
                         cudaMemcpyDeviceToHost, P.d2h) == cudaSuccess &&
         cudaMemcpy2DAsync(lse_h + t0, (size_t)T * 4, reinterpret_cast<float*>(w + off_l) + t0, (size_t)T * 4,
                           (size_t)(t1 - t0) * 4, (size_t)Hq, cudaMemcpyDeviceToHost, P.d2h) == cudaSuccess;
  }
  // everything this call queued has finished before it returns, also on an error
  const bool s1 = cudaStreamSynchronize(P.h2d) == cudaSuccess;
  const bool s2 = cudaStreamSynchronize(cs) == cudaSuccess;
  const bool s3 = cudaStreamSynchronize(P.d2h) == cudaSuccess;
  if (st != DAM_OK) return st;
  if (!ok || !s1 || !s2 || !s3) return DAM_ERR_CUDA;
  st = dam_poll_status(w + off_m, stream);
  if (st != DAM_OK) return st;
  return dam_poll_status(w + off_as, stream);
}

}  // extern "C"
