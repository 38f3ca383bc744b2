// C ABI of the SVD-Attention forward pass: argument checks, workspace layout,
// kernel selection.  Every host-visible error is returned before any launch.
#include <atomic>

#include "solar_internal.cuh"

namespace solar {
namespace {
std::atomic<int> g_slice_limit{0};     // solar_set_slice_limit
}  // namespace
int slice_limit() { return g_slice_limit.load(std::memory_order_relaxed); }
}  // namespace solar

using namespace solar;

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

solar_status_t check_dims(int B, int M, int N, int d, int r, solar_dtype_t dt) {
  if (dt != SOLAR_F32 && dt != SOLAR_BF16) return SOLAR_ERR_UNSUPPORTED;
  if (B < 0 || M < 0 || N < 1 || r < 1) return SOLAR_ERR_INVALID_ARG;
  if (d != 32 && d != 64 && d != 128) return SOLAR_ERR_UNSUPPORTED;
  if (r > d || r > N) return SOLAR_ERR_INVALID_ARG;
  if (r > 64 || B > 65535) return SOLAR_ERR_UNSUPPORTED;
  return SOLAR_OK;
}

solar_status_t check_ptr(const void* p) {
  return (p != nullptr && aligned16(p)) ? SOLAR_OK : SOLAR_ERR_INVALID_ARG;
}

solar_status_t check_ws(const void* ws, size_t have, size_t need) {
  if (ws == nullptr || !aligned16(ws) || have < need) return SOLAR_ERR_WORKSPACE;
  return SOLAR_OK;
}

#define SOLAR_TRY(expr)                       \
  do {                                        \
    const solar_status_t st__ = (expr);       \
    if (st__ != SOLAR_OK) return st__;        \
  } while (0)

solar_status_t from_cuda(cudaError_t e) { return e == cudaSuccess ? SOLAR_OK : SOLAR_ERR_CUDA; }

// Scores, softmax, weighted sum from a prepared workspace.  early_c: an earlier kernel of the
// same library call has already waited for whatever ran before the call, so the candidate tile
// may be fetched ahead of this kernel's own wait.
solar_status_t attn_apply_impl(int B, int M, int d, int r, solar_dtype_t dt, const void* C, unsigned flags,
                               void* O, const char* ws, bool early_c, cudaStream_t st) {
  if (attn_umma_supported(d, dt))
    return from_cuda(launch_attn_umma(B, M, d, r, C, flags, O, ws, attn_ws_layout(d, r), early_c, st));
  return from_cuda(launch_attn_simt(B, M, d, r, dt, C, flags, O, ws, attn_ws_layout(d, r), st));
}

// Workspace of the fused forward call: the factorization's, then the attention's.
size_t fused_attn_offset(int B, int N, int d, solar_dtype_t dt) { return align_up(factor_ws_bytes(B, N, d, dt), 256); }

}  // namespace

extern "C" {

const char* solar_status_string(solar_status_t st) {
  switch (st) {
    case SOLAR_OK: return "ok";
    case SOLAR_ERR_INVALID_ARG: return "invalid argument";
    case SOLAR_ERR_UNSUPPORTED: return "unsupported size, dtype or flag";
    case SOLAR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SOLAR_ERR_CUDA: return "CUDA error";
  }
  return "unknown status";
}

size_t solar_workspace_bytes(int B, int M, int N, int d, int r, solar_dtype_t dt) {
  if (check_dims(B, M, N, d, r, dt) != SOLAR_OK) return 0;
  const size_t f = factor_ws_bytes(B, N, d, dt), a = attn_ws_bytes(B, d, r);
  const size_t need = f > a ? f : a;
  return need ? need : 256;
}

int solar_set_slice_limit(int max_slices) {
  if (max_slices < 0) max_slices = 0;
  return solar::g_slice_limit.exchange(max_slices);
}

int solar_gram_splits(int B, int N, int d, solar_dtype_t dt) {
  if (check_dims(B, 0, N, d, 1, dt) != SOLAR_OK) return 0;
  return gram_plan(B, N, gram_is_clustered(N, d, dt)).parts;
}

int solar_gram_slices(int B, int N, int d, solar_dtype_t dt) {
  if (check_dims(B, 0, N, d, 1, dt) != SOLAR_OK) return 0;
  return gram_plan(B, N, gram_is_clustered(N, d, dt)).splits;
}

solar_status_t solar_gram_partials(int B, int N, int d, solar_dtype_t dt, const void* H,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  SOLAR_TRY(check_dims(B, 0, N, d, 1, dt));
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(H));
  SOLAR_TRY(check_ws(workspace, workspace_bytes, factor_ws_bytes(B, N, d, dt)));
  const GramPlan plan = gram_plan(B, N, gram_is_clustered(N, d, dt));
  float* gpart = static_cast<float*>(workspace);
  int* status = reinterpret_cast<int*>(static_cast<char*>(workspace) + gram_status_offset(B, N, d, dt));
  const cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (gram_umma_supported(N, d, dt)) return from_cuda(launch_gram_umma(B, N, d, H, gpart, status, plan, st));
  return from_cuda(launch_gram_simt(B, N, d, dt, H, gpart, status, plan, st));
}

solar_status_t solar_eig_from_partials_ex(int B, int N, int d, int r, solar_dtype_t dt, int route,
                                          float* S, float* V, int* info, int* route_taken,
                                          void* workspace, size_t workspace_bytes, void* stream) {
  SOLAR_TRY(check_dims(B, 0, N, d, r, dt));
  const int base_route = route & 0xff, sweep_cap = (route >> 8) & 0xff, force_iters = (route >> 16) & 0xff;
  if ((route & ~0xffffff) != 0 || base_route > SOLAR_ROUTE_TRIDIAG) return SOLAR_ERR_INVALID_ARG;
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  if (info != nullptr && (reinterpret_cast<uintptr_t>(info) & 3u)) return SOLAR_ERR_INVALID_ARG;
  if (route_taken != nullptr && (reinterpret_cast<uintptr_t>(route_taken) & 3u))
    return SOLAR_ERR_INVALID_ARG;
  SOLAR_TRY(check_ws(workspace, workspace_bytes, factor_ws_bytes(B, N, d, dt)));
  const GramPlan plan = gram_plan(B, N, gram_is_clustered(N, d, dt));
  const int* status =
      reinterpret_cast<const int*>(static_cast<const char*>(workspace) + gram_status_offset(B, N, d, dt));
  float* gsum = reinterpret_cast<float*>(static_cast<char*>(workspace) + gram_sum_offset(B, N, d, dt));
  return from_cuda(launch_eig(B, d, r, dt, base_route, sweep_cap, force_iters, static_cast<const float*>(workspace),
                              status, plan.parts, plan.splits, gsum, S, V, info, route_taken,
                              static_cast<cudaStream_t>(stream)));
}

solar_status_t solar_eig_from_partials(int B, int N, int d, int r, solar_dtype_t dt, float* S,
                                       float* V, int* info, void* workspace,
                                       size_t workspace_bytes, void* stream) {
  return solar_eig_from_partials_ex(B, N, d, r, dt, SOLAR_ROUTE_AUTO, S, V, info, nullptr,
                                    workspace, workspace_bytes, stream);
}

solar_status_t solar_project_us(int B, int N, int d, int r, solar_dtype_t dt, const void* H,
                                const float* V, void* US, void* stream) {
  SOLAR_TRY(check_dims(B, 0, N, d, r, dt));
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(H));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(US));
  return from_cuda(launch_project_us(B, N, d, r, dt, H, V, US, static_cast<cudaStream_t>(stream)));
}

solar_status_t solar_lowrank_factor(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                    const void* H, float* S, float* V, void* US, int* info,
                                    void* workspace, size_t workspace_bytes, void* stream) {
  (void)M;
  SOLAR_TRY(check_dims(B, 0, N, d, r, dt));
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(H));
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  if (US != nullptr) SOLAR_TRY(check_ptr(US));
  if (info != nullptr && (reinterpret_cast<uintptr_t>(info) & 3u)) return SOLAR_ERR_INVALID_ARG;
  SOLAR_TRY(check_ws(workspace, workspace_bytes, factor_ws_bytes(B, N, d, dt)));
  SOLAR_TRY(solar_gram_partials(B, N, d, dt, H, workspace, workspace_bytes, stream));
  SOLAR_TRY(solar_eig_from_partials(B, N, d, r, dt, S, V, info, workspace, workspace_bytes, stream));
  if (US != nullptr) SOLAR_TRY(solar_project_us(B, N, d, r, dt, H, V, US, stream));
  return SOLAR_OK;
}

solar_status_t solar_attn_prepare(int B, int d, int r, solar_dtype_t dt, const float* S,
                                  const float* V, const void* Wq, const void* Wk, const void* Wv,
                                  float scale, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  SOLAR_TRY(check_dims(B, 0, r, d, r, dt));
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(Wq));
  SOLAR_TRY(check_ptr(Wk));
  SOLAR_TRY(check_ptr(Wv));
  SOLAR_TRY(check_ws(workspace, workspace_bytes, attn_ws_bytes(B, d, r)));
  return from_cuda(launch_attn_prepare(B, d, r, dt, S, V, Wq, Wk, Wv, scale,
                                       static_cast<char*>(workspace), attn_ws_layout(d, r),
                                       static_cast<cudaStream_t>(stream)));
}

solar_status_t solar_attn_apply(int B, int M, int d, int r, solar_dtype_t dt, const void* C,
                                unsigned flags, void* O, void* workspace, size_t workspace_bytes,
                                void* stream) {
  SOLAR_TRY(check_dims(B, M, r, d, r, dt));
  if (flags & ~(unsigned)SOLAR_FLAG_NO_SOFTMAX) return SOLAR_ERR_UNSUPPORTED;
  if (B == 0 || M == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(C));
  SOLAR_TRY(check_ptr(O));
  SOLAR_TRY(check_ws(workspace, workspace_bytes, attn_ws_bytes(B, d, r)));
  return attn_apply_impl(B, M, d, r, dt, C, flags, O, static_cast<const char*>(workspace), false,
                         static_cast<cudaStream_t>(stream));
}

solar_status_t solar_svd_attention_fwd(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                       const void* C, const float* S, const float* V,
                                       const void* Wq, const void* Wk, const void* Wv, float scale,
                                       unsigned flags, void* O, void* workspace,
                                       size_t workspace_bytes, void* stream) {
  (void)N;
  SOLAR_TRY(check_dims(B, M, r, d, r, dt));
  if (flags & ~(unsigned)SOLAR_FLAG_NO_SOFTMAX) return SOLAR_ERR_UNSUPPORTED;
  if (B == 0 || M == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(C));
  SOLAR_TRY(check_ptr(O));
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(Wq));
  SOLAR_TRY(check_ptr(Wk));
  SOLAR_TRY(check_ptr(Wv));
  SOLAR_TRY(check_ws(workspace, workspace_bytes, attn_ws_bytes(B, d, r)));
  SOLAR_TRY(solar_attn_prepare(B, d, r, dt, S, V, Wq, Wk, Wv, scale, workspace, workspace_bytes,
                               stream));
  return attn_apply_impl(B, M, d, r, dt, C, flags, O, static_cast<const char*>(workspace), true,
                         static_cast<cudaStream_t>(stream));
}

size_t solar_fused_workspace_bytes(int B, int M, int N, int d, int r, solar_dtype_t dt) {
  if (check_dims(B, M, N, d, r, dt) != SOLAR_OK) return 0;
  return fused_attn_offset(B, N, d, dt) + align_up(attn_ws_bytes(B, d, r), 256);
}

solar_status_t solar_svd_attention_fused(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                         const void* H, const void* C, const void* Wq, const void* Wk,
                                         const void* Wv, float scale, unsigned flags, float* S, float* V,
                                         void* O, int* info, void* workspace, size_t workspace_bytes,
                                         void* stream) {
  SOLAR_TRY(check_dims(B, M, N, d, r, dt));
  if (flags & ~(unsigned)SOLAR_FLAG_NO_SOFTMAX) return SOLAR_ERR_UNSUPPORTED;
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(H));
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(Wq));
  SOLAR_TRY(check_ptr(Wk));
  SOLAR_TRY(check_ptr(Wv));
  if (M > 0) { SOLAR_TRY(check_ptr(C)); SOLAR_TRY(check_ptr(O)); }
  if (info != nullptr && (reinterpret_cast<uintptr_t>(info) & 3u)) return SOLAR_ERR_INVALID_ARG;
  SOLAR_TRY(check_ws(workspace, workspace_bytes, solar_fused_workspace_bytes(B, M, N, d, r, dt)));
  const cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  char* attn_ws = ws + fused_attn_offset(B, N, d, dt);
  // streaming pass over H (the first kernel of the call: it waits for what ran before)
  SOLAR_TRY(solar_gram_partials(B, N, d, dt, H, workspace, factor_ws_bytes(B, N, d, dt), stream));
  // eigensolve; every user's CTA ends with that user's factor-token projections
  const GramPlan plan = gram_plan(B, N, gram_is_clustered(N, d, dt));
  const int* status = reinterpret_cast<const int*>(ws + gram_status_offset(B, N, d, dt));
  float* gsum = reinterpret_cast<float*>(ws + gram_sum_offset(B, N, d, dt));
  const EigFuse fuse = {Wq, Wk, Wv, scale, attn_ws};
  SOLAR_TRY(from_cuda(launch_eig_tridiag(B, d, r, dt, SOLAR_ROUTE_AUTO, kMaxSweeps, reinterpret_cast<const float*>(ws),
                                         status, plan.parts, plan.splits, gsum, S, V, info, nullptr, &fuse, st)));
  if (M == 0) return SOLAR_OK;
  return attn_apply_impl(B, M, d, r, dt, C, flags, O, attn_ws, true, st);
}

size_t solar_backward_workspace_bytes(int B, int M, int N, int d, int r, solar_dtype_t dt) {
  if (check_dims(B, M, N, d, r, dt) != SOLAR_OK) return 0;
  const size_t a = bwd_ws_layout(B, M, d, r).total, k = (size_t)B * d * d * sizeof(float);
  return a > k ? a : k;
}

solar_status_t solar_svd_attention_bwd(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                       const void* C, const float* S, const float* V,
                                       const void* Wq, const void* Wk, const void* Wv,
                                       float scale, unsigned flags, const void* dO,
                                       void* dC, float* dWq, float* dWk, float* dWv,
                                       float* dS, float* dV,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  (void)N;
  SOLAR_TRY(check_dims(B, M, r, d, r, dt));
  if (flags & ~(unsigned)SOLAR_FLAG_NO_SOFTMAX) return SOLAR_ERR_UNSUPPORTED;
  if (B == 0) return SOLAR_OK;
  if (M > 0) { SOLAR_TRY(check_ptr(C)); SOLAR_TRY(check_ptr(dO)); SOLAR_TRY(check_ptr(dC)); }
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(Wq));
  SOLAR_TRY(check_ptr(Wk));
  SOLAR_TRY(check_ptr(Wv));
  SOLAR_TRY(check_ptr(dWq));
  SOLAR_TRY(check_ptr(dWk));
  SOLAR_TRY(check_ptr(dWv));
  SOLAR_TRY(check_ptr(dS));
  SOLAR_TRY(check_ptr(dV));
  const BwdWs bl = bwd_ws_layout(B, M, d, r);
  SOLAR_TRY(check_ws(workspace, workspace_bytes, bl.total));
  const cudaStream_t st = static_cast<cudaStream_t>(stream);
  const AttnWs lay = attn_ws_layout(d, r);
  char* ws = static_cast<char*>(workspace);
  // T_b and Value_r as in the forward call
  SOLAR_TRY(from_cuda(launch_attn_prepare(B, d, r, dt, S, V, Wq, Wk, Wv, scale, ws, lay, st)));
  return from_cuda(launch_attn_bwd(B, M, d, r, dt, C, dO, S, V, Wq, Wk, Wv, scale, flags, dC, dWq, dWk, dWv,
                                   dS, dV, ws, lay, bl, st));
}

solar_status_t solar_svd_backward(int B, int N, int d, int r, solar_dtype_t dt, const void* H,
                                  const float* S, const float* V, const float* dS, const float* dV,
                                  float eps_rel, void* dH, void* workspace, size_t workspace_bytes,
                                  void* stream) {
  SOLAR_TRY(check_dims(B, 0, N, d, r, dt));
  if (!(eps_rel >= 0.f)) return SOLAR_ERR_INVALID_ARG;
  if (B == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(H));
  SOLAR_TRY(check_ptr(S));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(dS));
  SOLAR_TRY(check_ptr(dV));
  SOLAR_TRY(check_ptr(dH));
  SOLAR_TRY(check_ws(workspace, workspace_bytes, (size_t)B * d * d * sizeof(float)));
  const cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* K = static_cast<float*>(workspace);
  SOLAR_TRY(from_cuda(launch_svd_grad(B, d, r, S, V, dS, dV, eps_rel, K, st)));
  // dH_b = H_b K_b: the right-multiplication kernel of the left factor, with q = d columns
  return from_cuda(launch_project_us(B, N, d, d, dt, H, K, dH, st));
}

solar_status_t solar_factored_softmax_attention_fwd(int B, int M, int N, int d, int r, solar_dtype_t dt,
                                                    const void* C, const void* US, const float* V,
                                                    const void* Wq, const void* Wk, const void* Wv,
                                                    float scale, void* O, void* workspace,
                                                    size_t workspace_bytes, void* stream) {
  SOLAR_TRY(check_dims(B, M, N, d, r, dt));
  if (!flash_factored_supported(d, r, dt)) return SOLAR_ERR_UNSUPPORTED;
  if (B == 0 || M == 0) return SOLAR_OK;
  SOLAR_TRY(check_ptr(C));
  SOLAR_TRY(check_ptr(US));
  SOLAR_TRY(check_ptr(V));
  SOLAR_TRY(check_ptr(Wq));
  SOLAR_TRY(check_ptr(Wk));
  SOLAR_TRY(check_ptr(Wv));
  SOLAR_TRY(check_ptr(O));
  SOLAR_TRY(check_ws(workspace, workspace_bytes, attn_ws_bytes(B, d, r)));
  const cudaStream_t st = static_cast<cudaStream_t>(stream);
  const AttnWs lay = attn_ws_layout(d, r);
  // The packed operands of the kernel are the prepare kernel's with unit singular values:
  // T^T becomes (scale log2e W_Q W_K^T V)^T and Value_r^T becomes (V^T W_V)^T.
  SOLAR_TRY(from_cuda(launch_attn_prepare(B, d, r, dt, nullptr, V, Wq, Wk, Wv,
                                          scale * 1.4426950408889634f, static_cast<char*>(workspace), lay, st)));
  return from_cuda(launch_flash_factored(B, M, N, d, r, C, US, O, static_cast<const char*>(workspace), lay, st));
}

}  // extern "C"
