// extern "C" entry points of the kvcrush library: argument validation and stage dispatch.
// Every check that can fail happens before the first launch, so an error return means nothing ran.
#include <math.h>

#include "common.cuh"

namespace {

using namespace kvc;

constexpr size_t kAlign = 256;
inline size_t round_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

int make_shape(const kvcrush_problem_t* p, Shape* s) {
  if (!p) return KVCRUSH_ERR_INVALID_ARG;
  if (p->n_layers < 1 || p->n_seqs < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->head_dim < 1 ||
      p->total_tokens < 0 || p->max_seqlen < 0 || p->query_window < 0)
    return KVCRUSH_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return KVCRUSH_ERR_INVALID_ARG;
  if (p->n_q_heads > 128) return KVCRUSH_ERR_UNSUPPORTED;
  if (!p->cu_seqlens_host || !p->cu_seqlens_dev) return KVCRUSH_ERR_INVALID_ARG;
  const int32_t* cu = p->cu_seqlens_host;
  if (cu[0] != 0 || cu[p->n_seqs] != p->total_tokens) return KVCRUSH_ERR_INVALID_ARG;
  for (int i = 0; i < p->n_seqs; ++i) {
    const int len = cu[i + 1] - cu[i];
    if (len < 0 || len > p->max_seqlen) return KVCRUSH_ERR_INVALID_ARG;
  }
  if ((long long)p->n_layers * p->n_q_heads * (long long)p->total_tokens > (1LL << 40)) return KVCRUSH_ERR_UNSUPPORTED;
  s->n_layers = p->n_layers; s->n_seqs = p->n_seqs; s->Hq = p->n_q_heads; s->Hkv = p->n_kv_heads;
  s->D = p->head_dim; s->T = p->total_tokens; s->max_seqlen = p->max_seqlen; s->causal = p->causal != 0;
  s->G = p->n_q_heads / p->n_kv_heads; s->W = (p->n_q_heads + 31) / 32;
  s->cu_seqlens = p->cu_seqlens_dev;
  s->window = p->query_window;
  return KVCRUSH_OK;
}

int make_view(const kvcrush_tensor_t* t, int head_dim, TensorView* v) {
  if (!t || !t->ptr_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (t->dtype != KVCRUSH_BF16 && t->dtype != KVCRUSH_FP16 && t->dtype != KVCRUSH_FP32) return KVCRUSH_ERR_INVALID_ARG;
  const int eb = elt_bytes(t->dtype);
  if (reinterpret_cast<uintptr_t>(t->ptr_dev) % 16 != 0) return KVCRUSH_ERR_MISALIGNED;
  if ((t->stride_layer * eb) % 16 || (t->stride_token * eb) % 16 || (t->stride_head * eb) % 16 ||
      ((long long)head_dim * eb) % 16)
    return KVCRUSH_ERR_MISALIGNED;
  if (t->stride_layer < 0 || t->stride_token < 0 || t->stride_head < 0) return KVCRUSH_ERR_INVALID_ARG;
  v->ptr = t->ptr_dev; v->dtype = t->dtype; v->sl = t->stride_layer; v->st = t->stride_token; v->sh = t->stride_head;
  return KVCRUSH_OK;
}

size_t score_lse_bytes(const Shape& s) { return round_up((size_t)s.n_layers * s.Hq * s.T * sizeof(float)); }
// work counters of the persistent tensor-core kernels first, then the row log-sum-exp of every query
size_t score_counter_bytes() { return round_up(score_tensor_counter_bytes()); }
size_t score_ws(const Shape& s) { return score_counter_bytes() + score_lse_bytes(s); }
size_t signature_ws(const Shape& s) { return round_up((size_t)s.n_layers * s.n_seqs * s.Hq * sizeof(float)); }

}  // namespace

namespace kvc {
int shape_from_problem(const kvcrush_problem_t* problem, Shape* out) { return make_shape(problem, out); }
}  // namespace kvc

extern "C" {

int kvcrush_workspace_size(const kvcrush_problem_t* problem, int stage, size_t* bytes) {
  Shape s;
  if (!bytes) return KVCRUSH_ERR_INVALID_ARG;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  switch (stage) {
    case KVCRUSH_STAGE_SCORE: *bytes = score_ws(s); return KVCRUSH_OK;
    case KVCRUSH_STAGE_SIGNATURE: *bytes = signature_ws(s); return KVCRUSH_OK;
    case KVCRUSH_STAGE_SELECT: *bytes = select_workspace_bytes(s); return KVCRUSH_OK;
    case KVCRUSH_STAGE_COMPACT: *bytes = 0; return KVCRUSH_OK;
    default: return KVCRUSH_ERR_INVALID_ARG;
  }
}

}  // extern "C"

namespace {

int score_entry(const kvcrush_problem_t* problem, const kvcrush_tensor_t* Q, const kvcrush_tensor_t* K,
                const float* lse_in_dev, float* scores_dev, float* lse_out_dev, int normalize, int impl,
                void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream, const ScoreDiag& diag) {
  Shape s;
  int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  TensorView q, k;
  if ((rc = make_view(Q, s.D, &q)) != KVCRUSH_OK) return rc;
  if ((rc = make_view(K, s.D, &k)) != KVCRUSH_OK) return rc;
  if (!scores_dev || !status_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (q.dtype != k.dtype) return KVCRUSH_ERR_INVALID_ARG;
  if (impl != KVCRUSH_SCORE_AUTO && impl != KVCRUSH_SCORE_SIMT && impl != KVCRUSH_SCORE_TENSOR)
    return KVCRUSH_ERR_INVALID_ARG;
  // with the row log-sum-exp supplied only the work counters live in the workspace
  if (!workspace || workspace_bytes < (lse_in_dev ? score_counter_bytes() : score_ws(s))) return KVCRUSH_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return KVCRUSH_ERR_MISALIGNED;
  int* counters = static_cast<int*>(workspace);
  float* lse2_ws = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + score_counter_bytes());
  const float scale = problem->softmax_scale != 0.f ? problem->softmax_scale : 1.f / sqrtf((float)s.D);
  const float log2e = 1.4426950408889634f;
  const float scale_log2 = scale * log2e;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ScoreTensorMaps maps;
  const int plan = impl == KVCRUSH_SCORE_SIMT ? TENSOR_PLAN_NO : score_tensor_plan(s, q, k, &maps);
  // a problem made for the tensor cores must not end up on the CUDA cores because the driver lacks the encoder
  if (plan == TENSOR_PLAN_NO_ENCODER) return KVCRUSH_ERR_UNSUPPORTED;
  if (plan == TENSOR_PLAN_NO) {
    if (impl == KVCRUSH_SCORE_TENSOR) return KVCRUSH_ERR_UNSUPPORTED;
    return launch_score_simt(s, q, k, scale_log2, lse_in_dev, log2e, lse2_ws, scores_dev, lse_out_dev, normalize,
                             status_dev, st);
  }
  return launch_score_tensor(s, problem->cu_seqlens_host, q, maps, scale_log2, lse_in_dev, log2e, lse2_ws, counters,
                             scores_dev, lse_out_dev, normalize, status_dev, diag, st);
}

}  // namespace

extern "C" {

int kvcrush_score(const kvcrush_problem_t* problem, const kvcrush_tensor_t* Q, const kvcrush_tensor_t* K,
                  const float* lse_in_dev, float* scores_dev, float* lse_out_dev, int normalize, int impl,
                  void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  return score_entry(problem, Q, K, lse_in_dev, scores_dev, lse_out_dev, normalize, impl, workspace, workspace_bytes,
                     status_dev, stream, ScoreDiag{});
}

// Not part of the public ABI (the header does not declare it): kvcrush_score with the diagnostics of the tensor-core
// kernels exposed, for the test that makes a bounded wait run out.  short_waits != 0 runs the instantiation of the
// kernels whose barrier waits give up after a few thousand polls; withhold_first_item != 0 makes the producer warp of
// every CTA stop after fetching its first work item, before announcing it and before issuing any copy, so that the
// other roles' first waits run out with nothing in flight: the kernels return normally with
// status = {KVCRUSH_DEV_TIMEOUT, kernel id, block, 0}.
int kvcrush_diag_score(const kvcrush_problem_t* problem, const kvcrush_tensor_t* Q, const kvcrush_tensor_t* K,
                       const float* lse_in_dev, float* scores_dev, float* lse_out_dev, int normalize, int impl,
                       void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream,
                       int short_waits, int withhold_first_item) {
  ScoreDiag diag{};
  diag.short_waits = short_waits != 0;
  diag.withhold_first_item = withhold_first_item != 0;
  return score_entry(problem, Q, K, lse_in_dev, scores_dev, lse_out_dev, normalize, impl, workspace, workspace_bytes,
                     status_dev, stream, diag);
}

int kvcrush_score_decode(const kvcrush_problem_t* problem, const kvcrush_tensor_t* Q_new, const kvcrush_tensor_t* K,
                         float* scores_dev, int32_t* status_dev, void* stream) {
  Shape s;
  int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  TensorView q, k;
  if ((rc = make_view(Q_new, s.D, &q)) != KVCRUSH_OK) return rc;
  if ((rc = make_view(K, s.D, &k)) != KVCRUSH_OK) return rc;
  if (!scores_dev || !status_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (q.dtype != k.dtype) return KVCRUSH_ERR_INVALID_ARG;
  const float scale = problem->softmax_scale != 0.f ? problem->softmax_scale : 1.f / sqrtf((float)s.D);
  return launch_score_decode(s, q, k, scale * 1.4426950408889634f, scores_dev, static_cast<cudaStream_t>(stream));
}

int kvcrush_signature(const kvcrush_problem_t* problem, const float* scores_dev, const int32_t* sig_keep_dev,
                      const float* theta_in_dev, uint32_t* sigs_dev, float* theta_out_dev, double* importance_out_dev,
                      void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  Shape s;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if (!scores_dev || !sigs_dev || !status_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (!theta_in_dev && !sig_keep_dev) return KVCRUSH_ERR_INVALID_ARG;
  float* theta = theta_out_dev;
  if (!theta_in_dev && !theta) {
    if (!workspace || workspace_bytes < signature_ws(s)) return KVCRUSH_ERR_WORKSPACE;
    theta = static_cast<float*>(workspace);
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (theta_in_dev && theta_out_dev && theta_out_dev != theta_in_dev) {
    if (cudaMemcpyAsync(theta_out_dev, theta_in_dev, (size_t)s.n_layers * s.n_seqs * s.Hq * sizeof(float),
                        cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return KVCRUSH_ERR_CUDA;
  }
  if (importance_out_dev && reinterpret_cast<uintptr_t>(importance_out_dev) % 8) return KVCRUSH_ERR_MISALIGNED;
  return launch_signature(s, scores_dev, sig_keep_dev, theta_in_dev, sigs_dev, theta, importance_out_dev, st);
}

int kvcrush_select(const kvcrush_problem_t* problem, const float* scores_dev, const double* importance_dev,
                   const uint32_t* sigs_dev, const int32_t* budget_imp_dev, const int32_t* budget_rep_dev,
                   int anchor_mode, const uint32_t* anchor_bits_dev, int anchor_per_segment,
                   int keep_initial, int keep_recent,
                   const int32_t* cu_kept_dev, int32_t* idx_dev, uint8_t* kind_dev, int32_t* n_kept_dev,
                   void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  Shape s;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if ((!scores_dev && !importance_dev) || !sigs_dev || !budget_imp_dev || !budget_rep_dev || !cu_kept_dev || !idx_dev ||
      !status_dev)
    return KVCRUSH_ERR_INVALID_ARG;
  if (importance_dev && reinterpret_cast<uintptr_t>(importance_dev) % 8) return KVCRUSH_ERR_MISALIGNED;
  if (anchor_mode != KVCRUSH_ANCHOR_ALTERNATE && anchor_mode != KVCRUSH_ANCHOR_MEAN &&
      anchor_mode != KVCRUSH_ANCHOR_EXPLICIT)
    return KVCRUSH_ERR_INVALID_ARG;
  if (anchor_mode == KVCRUSH_ANCHOR_EXPLICIT && !anchor_bits_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (keep_recent < 0 || keep_initial < 0) return KVCRUSH_ERR_INVALID_ARG;
  if (s.max_seqlen > 262144) return KVCRUSH_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < select_workspace_bytes(s)) return KVCRUSH_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return KVCRUSH_ERR_MISALIGNED;
  return launch_select(s, scores_dev, importance_dev, sigs_dev, budget_imp_dev, budget_rep_dev, anchor_mode, anchor_bits_dev,
                       anchor_per_segment != 0, keep_initial, keep_recent, cu_kept_dev, idx_dev, kind_dev, n_kept_dev,
                       workspace, static_cast<cudaStream_t>(stream));
}

int kvcrush_kmeans_workspace_size(const kvcrush_problem_t* problem, int max_budget_rep, size_t* bytes) {
  Shape s;
  if (!bytes || max_budget_rep < 0) return KVCRUSH_ERR_INVALID_ARG;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  *bytes = kmeans_workspace_bytes(s, max_budget_rep);
  return KVCRUSH_OK;
}

int kvcrush_kmeans_select(const kvcrush_problem_t* problem, const float* scores_dev, const double* importance_dev,
                          const uint32_t* sigs_dev, const int32_t* budget_imp_dev, const int32_t* budget_rep_dev,
                          int max_budget_rep, int iterations, int keep_initial, int keep_recent,
                          const int32_t* cu_kept_dev, int32_t* idx_dev, uint8_t* kind_dev, int32_t* n_kept_dev,
                          void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  Shape s;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if ((!scores_dev && !importance_dev) || !sigs_dev || !budget_imp_dev || !budget_rep_dev || !cu_kept_dev || !idx_dev ||
      !status_dev)
    return KVCRUSH_ERR_INVALID_ARG;
  if (importance_dev && reinterpret_cast<uintptr_t>(importance_dev) % 8) return KVCRUSH_ERR_MISALIGNED;
  if (max_budget_rep < 0 || iterations < 0 || keep_recent < 0 || keep_initial < 0) return KVCRUSH_ERR_INVALID_ARG;
  if (!kmeans_supported(s)) return KVCRUSH_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < kmeans_workspace_bytes(s, max_budget_rep)) return KVCRUSH_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return KVCRUSH_ERR_MISALIGNED;
  return launch_kmeans_select(s, scores_dev, importance_dev, sigs_dev, budget_imp_dev, budget_rep_dev, max_budget_rep,
                              iterations, keep_initial, keep_recent, cu_kept_dev, idx_dev, kind_dev, n_kept_dev,
                              workspace, status_dev, static_cast<cudaStream_t>(stream));
}

int kvcrush_compact(const kvcrush_problem_t* problem, const kvcrush_tensor_t* K, const kvcrush_tensor_t* V,
                    const int32_t* cu_kept_dev, const int32_t* idx_dev, int64_t total_kept,
                    const kvcrush_tensor_t* K_out, const kvcrush_tensor_t* V_out,
                    int32_t* status_dev, void* stream) {
  Shape s;
  int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if (!cu_kept_dev || !idx_dev || !status_dev || total_kept < 0) return KVCRUSH_ERR_INVALID_ARG;
  if ((V == nullptr) != (V_out == nullptr)) return KVCRUSH_ERR_INVALID_ARG;
  TensorView k, v, ko, vo;
  if ((rc = make_view(K, s.D, &k)) != KVCRUSH_OK) return rc;
  if ((rc = make_view(K_out, s.D, &ko)) != KVCRUSH_OK) return rc;
  if (k.dtype != ko.dtype) return KVCRUSH_ERR_INVALID_ARG;
  if (V) {
    if ((rc = make_view(V, s.D, &v)) != KVCRUSH_OK) return rc;
    if ((rc = make_view(V_out, s.D, &vo)) != KVCRUSH_OK) return rc;
    if (v.dtype != k.dtype || vo.dtype != k.dtype) return KVCRUSH_ERR_INVALID_ARG;
  }
  return launch_compact(s, k, V ? &v : nullptr, cu_kept_dev, idx_dev, total_kept, ko, V ? &vo : nullptr,
                        static_cast<cudaStream_t>(stream));
}

int kvcrush_select_pages(const kvcrush_problem_t* problem, const float* scores_dev, const double* importance_dev,
                         const uint32_t* sigs_dev, int page_size, const int32_t* budget_imp_dev, const int32_t* budget_rep_dev,
                         int anchor_mode, const uint32_t* anchor_bits_dev, int anchor_per_segment,
                         int keep_initial, int keep_recent,
                         const int32_t* cu_kept_dev, int32_t* page_idx_dev, uint8_t* kind_dev, int32_t* n_kept_dev,
                         void* workspace, size_t workspace_bytes, int32_t* status_dev, void* stream) {
  Shape s;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if ((!scores_dev && !importance_dev) || !sigs_dev || !budget_imp_dev || !budget_rep_dev || !cu_kept_dev ||
      !page_idx_dev || !status_dev)
    return KVCRUSH_ERR_INVALID_ARG;
  if (importance_dev && reinterpret_cast<uintptr_t>(importance_dev) % 8) return KVCRUSH_ERR_MISALIGNED;
  if (anchor_mode != KVCRUSH_ANCHOR_ALTERNATE && anchor_mode != KVCRUSH_ANCHOR_MEAN &&
      anchor_mode != KVCRUSH_ANCHOR_EXPLICIT)
    return KVCRUSH_ERR_INVALID_ARG;
  if (anchor_mode == KVCRUSH_ANCHOR_EXPLICIT && !anchor_bits_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (page_size < 1 || keep_initial < 0 || keep_recent < 0) return KVCRUSH_ERR_INVALID_ARG;
  if ((long long)page_size * s.W > kMaxPageWords) return KVCRUSH_ERR_UNSUPPORTED;
  if (((long long)s.max_seqlen + page_size - 1) / page_size > kMaxPagesPerSeq) return KVCRUSH_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < select_workspace_bytes(s)) return KVCRUSH_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign) return KVCRUSH_ERR_MISALIGNED;
  return launch_select_pages(s, scores_dev, importance_dev, sigs_dev, page_size, budget_imp_dev, budget_rep_dev, anchor_mode,
                             anchor_bits_dev, anchor_per_segment != 0, keep_initial, keep_recent, cu_kept_dev,
                             page_idx_dev, kind_dev, n_kept_dev,
                             workspace, static_cast<cudaStream_t>(stream));
}

int kvcrush_compact_pages(const kvcrush_problem_t* problem, const kvcrush_tensor_t* K, const kvcrush_tensor_t* V,
                          int page_size, const int32_t* cu_kept_dev, const int32_t* page_idx_dev,
                          int64_t total_kept_pages, const kvcrush_tensor_t* K_out, const kvcrush_tensor_t* V_out,
                          int32_t* status_dev, void* stream) {
  Shape s;
  int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if (!cu_kept_dev || !page_idx_dev || !status_dev || total_kept_pages < 0 || page_size < 1)
    return KVCRUSH_ERR_INVALID_ARG;
  if ((V == nullptr) != (V_out == nullptr)) return KVCRUSH_ERR_INVALID_ARG;
  TensorView k, v, ko, vo;
  if ((rc = make_view(K, s.D, &k)) != KVCRUSH_OK) return rc;
  if ((rc = make_view(K_out, s.D, &ko)) != KVCRUSH_OK) return rc;
  if (k.dtype != ko.dtype) return KVCRUSH_ERR_INVALID_ARG;
  if (V) {
    if ((rc = make_view(V, s.D, &v)) != KVCRUSH_OK) return rc;
    if ((rc = make_view(V_out, s.D, &vo)) != KVCRUSH_OK) return rc;
    if (v.dtype != k.dtype || vo.dtype != k.dtype) return KVCRUSH_ERR_INVALID_ARG;
  }
  return launch_compact_pages(s, k, V ? &v : nullptr, page_size, cu_kept_dev, page_idx_dev, total_kept_pages, ko,
                              V ? &vo : nullptr, static_cast<cudaStream_t>(stream));
}

int kvcrush_compact_scores(const kvcrush_problem_t* problem, const float* scores_in_dev, int page_size,
                           const int32_t* cu_kept_dev, const int32_t* idx_dev, int64_t total_kept,
                           float* scores_out_dev, int64_t out_tokens, int32_t* status_dev, void* stream) {
  Shape s;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if (!scores_in_dev || !scores_out_dev || scores_in_dev == scores_out_dev || !cu_kept_dev || !idx_dev || !status_dev)
    return KVCRUSH_ERR_INVALID_ARG;
  if (page_size < 0 || total_kept < 0 || out_tokens < 0) return KVCRUSH_ERR_INVALID_ARG;
  return launch_compact_scores(s, scores_in_dev, page_size, cu_kept_dev, idx_dev, total_kept, scores_out_dev,
                               out_tokens, static_cast<cudaStream_t>(stream));
}

int kvcrush_pool_scores(const kvcrush_problem_t* problem, const float* scores_in_dev, int kernel,
                        float* scores_out_dev, int32_t* status_dev, void* stream) {
  Shape s;
  const int rc = make_shape(problem, &s);
  if (rc != KVCRUSH_OK) return rc;
  if (!scores_in_dev || !scores_out_dev || !status_dev || scores_in_dev == scores_out_dev) return KVCRUSH_ERR_INVALID_ARG;
  if (kernel < 1 || kernel % 2 == 0) return KVCRUSH_ERR_INVALID_ARG;
  return launch_pool_scores(s, scores_in_dev, kernel, scores_out_dev, static_cast<cudaStream_t>(stream));
}

const char* kvcrush_strerror(int code) {
  switch (code) {
    case KVCRUSH_OK: return "ok";
    case KVCRUSH_ERR_INVALID_ARG: return "invalid argument";
    case KVCRUSH_ERR_UNSUPPORTED: return "unsupported shape or type";
    case KVCRUSH_ERR_MISALIGNED: return "misaligned pointer or stride";
    case KVCRUSH_ERR_WORKSPACE: return "workspace missing or too small";
    case KVCRUSH_ERR_CUDA: return "CUDA call failed";
    case KVCRUSH_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch array";
    default: return "unknown error";
  }
}

int kvcrush_version(void) { return 100; }

}  // extern "C"
