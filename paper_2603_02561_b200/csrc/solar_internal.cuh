// Internal declarations shared by the kernels of the SVD-Attention forward pass.
// Nothing here is part of the C ABI (include/solar.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "solar.h"

namespace solar {

constexpr int kNumSMs = 148;        // B200: 2 dies x 74 SMs
constexpr int kGramTileRows = 128;  // rows of H per streamed tile
constexpr int kMaxSplits = 64;
constexpr int kMaxSweeps = 16;      // Jacobi sweep cap

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline size_t elem_size(solar_dtype_t dt) { return dt == SOLAR_BF16 ? 2 : 4; }

// How each H_b is cut into row slices for a streaming pass (one CTA per user and slice).  The
// cost model is waves(B*S CTAs over the SMs) x (tiles per slice + fixed per-CTA cost).
struct GramPlan {
  int tiles;        // ceil(N / kGramTileRows)
  int chunk_tiles;  // tiles per slice
  int splits;       // slices per user (all non-empty)
  int cluster;      // slices whose CTAs form one thread-block cluster and add up their results on chip
  int parts;        // partial Gram matrices per user that reach global memory: splits / cluster
};

inline long slice_cost(int B, int tiles, int s, int* s_eff_out, int* chunk_out) {
  const int chunk = (tiles + s - 1) / s;
  const int s_eff = (tiles + chunk - 1) / chunk;
  const long waves = ((long)B * s_eff + kNumSMs - 1) / kNumSMs;
  *s_eff_out = s_eff; *chunk_out = chunk;
  return waves * (chunk + 2);
}

// Process-wide cap on the slices per user (solar_set_slice_limit; 0 = none).
int slice_limit();

inline GramPlan slice_plan(int B, int N) {
  GramPlan p;
  p.tiles = (N + kGramTileRows - 1) / kGramTileRows;
  long best_cost = -1;
  int smax = p.tiles < kMaxSplits ? p.tiles : kMaxSplits;
  const int cap = slice_limit();
  if (cap > 0 && cap < smax) smax = cap;
  p.splits = 1; p.chunk_tiles = p.tiles;
  for (int s = 1; s <= smax; ++s) {
    int s_eff, chunk;
    const long cost = slice_cost(B, p.tiles, s, &s_eff, &chunk);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; p.splits = s_eff; p.chunk_tiles = chunk; }
  }
  p.cluster = 1;
  p.parts = p.splits;
  return p;
}

// The plan of the tensor-core Gram kernel.  Its CTAs can form thread-block clusters of
// kMaxCluster slices of a user that add up their accumulators through distributed shared
// memory, so that a user leaves splits / cluster partial matrices.  Measured on the headline
// shape (B = 16, N = 10240: nine slices), clusters of 3 and of 8 both lose more in the Gram
// kernel (gang-scheduled CTAs, two cluster barriers: 3.3 -> 3.95 us per launch with 24 requests
// in flight, 7.4 -> 9.9 us alone) than the eigensolver gains from reading one matrix instead
// of nine (45 -> 44 us), so the cluster size is 1 and every slice writes its own partial.
constexpr int kMaxCluster = 1;
inline GramPlan gram_plan(int B, int N, bool clustered) {
  if (!clustered) return slice_plan(B, N);
  GramPlan p;
  p.tiles = (N + kGramTileRows - 1) / kGramTileRows;
  long best_cost = -1;
  int smax = p.tiles < kMaxSplits ? p.tiles : kMaxSplits;
  const int cap = slice_limit();
  if (cap > 0 && cap < smax) smax = cap;
  p.splits = 1; p.chunk_tiles = p.tiles;
  for (int s = 1; s <= smax; ++s) {
    int s_eff, chunk;
    const long cost = slice_cost(B, p.tiles, s, &s_eff, &chunk);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; p.splits = s_eff; p.chunk_tiles = chunk; }
  }
  // the largest cluster size (<= kMaxCluster) that divides the slice count
  p.cluster = 1;
  for (int c = 2; c <= kMaxCluster; ++c)
    if (p.splits % c == 0) p.cluster = c;
  p.parts = p.splits / p.cluster;
  return p;
}
inline bool gram_is_clustered(int N, int d, solar_dtype_t dt) {
  return dt == SOLAR_BF16 && (d == 64 || d == 128) && N >= kGramTileRows;   // the tensor-core kernel's shapes
}

// Workspace of the factorization: partial Grams [B][parts][d][d] fp32, then one status word per
// (user, slice), written by every Gram CTA: kGramStatusOk, or the code of the bounded
// device-side wait that ran out.
constexpr int kGramStatusOk = 0x600D;
inline size_t gram_status_offset(int B, int N, int d, solar_dtype_t dt) {
  const GramPlan p = gram_plan(B, N, gram_is_clustered(N, d, dt));
  return align_up((size_t)B * p.parts * d * d * sizeof(float), 256);
}
// Behind the status words: the summed Gram matrices [B][d][d] fp32, written by the eigensolver
// when a user has more than one partial (its residual check and its Jacobi fallback read the
// sum back; a single partial is the sum).
inline size_t gram_sum_offset(int B, int N, int d, solar_dtype_t dt) {
  const GramPlan p = gram_plan(B, N, gram_is_clustered(N, d, dt));
  return gram_status_offset(B, N, d, dt) + align_up((size_t)B * p.splits * sizeof(int), 256);
}
inline size_t factor_ws_bytes(int B, int N, int d, solar_dtype_t dt) {
  return gram_sum_offset(B, N, d, dt) + align_up((size_t)B * d * d * sizeof(float), 256);
}

// Workspace of the attention call, per user (all segments 256-byte aligned):
//   Tf   [d][r]      fp32  folded score operand  scale * W_Q Key_r^T
//   Vr   [r][d]      fp32  Value_r
//   Tpk  [2][64][d]  bf16  T^T split into a high and a low bf16 half (rows >= r are zero):
//                          the score GEMM's B operand, K-major, for the tensor-core kernel
//   Vpk  [2][d][64]  bf16  Value_r^T, high and low halves (columns >= r are zero):
//                          the output GEMM's B operand, K-major
constexpr int kTokenSlots = 64;     // r <= 64 factor tokens, zero padded in the packed operands
struct AttnWs {
  size_t tf_off, vr_off, tpk_off, vpk_off, per_user;
};
inline AttnWs attn_ws_layout(int d, int r) {
  AttnWs w;
  size_t o = 0;
  w.tf_off = o;  o += align_up((size_t)d * r * 4, 256);
  w.vr_off = o;  o += align_up((size_t)d * r * 4, 256);
  w.tpk_off = o; o += align_up((size_t)2 * kTokenSlots * d * 2, 256);
  w.vpk_off = o; o += align_up((size_t)2 * d * kTokenSlots * 2, 256);
  w.per_user = o;
  return w;
}
inline size_t attn_ws_bytes(int B, int d, int r) {
  return attn_ws_layout(d, r).per_user * (size_t)B;
}

// Backward pass of the attention: how the M candidates of a user are cut into row chunks
// (one CTA each; every chunk leaves one partial of the two per-user reductions over M),
// and the workspace behind the attention call's own segments:
//   part [B][chunks][2][d][64] fp32   partial dT (= C^T dS) and dValue_r^T (= dO^T P)
//   dw   [B][3][d][d]          fp32   per-user contributions to dW_Q, dW_K, dW_V
struct BwdPlan {
  int rows_per_cta;   // a multiple of 32
  int chunks;
};
inline BwdPlan bwd_plan(int B, int M) {
  BwdPlan p;
  const int b = B > 0 ? B : 1;
  int want = (2 * kNumSMs + b - 1) / b;               // about two CTAs per SM over all users
  const int max_chunks = (M + 31) / 32 > 0 ? (M + 31) / 32 : 1;
  if (want > max_chunks) want = max_chunks;
  if (want < 1) want = 1;
  p.rows_per_cta = (((M + want - 1) / want + 31) / 32) * 32;
  if (p.rows_per_cta < 32) p.rows_per_cta = 32;
  p.chunks = (M + p.rows_per_cta - 1) / p.rows_per_cta;
  if (p.chunks < 1) p.chunks = 1;
  return p;
}
// The tensor-core kernel works on whole 128-row tiles: tiles per CTA and the number of chunks.
struct BwdTilePlan {
  int tiles_per_cta, chunks;
};
inline BwdTilePlan bwd_tile_plan(int B, int M) {
  BwdTilePlan p;
  const int b = B > 0 ? B : 1;
  const int tiles = (M + 127) / 128 > 0 ? (M + 127) / 128 : 1;
  int want = (2 * kNumSMs + b - 1) / b;
  if (want > tiles) want = tiles;
  p.tiles_per_cta = (tiles + want - 1) / want;
  p.chunks = (tiles + p.tiles_per_cta - 1) / p.tiles_per_cta;
  return p;
}
//   pk   [B][4][64][d]         bf16   T and Value_r as the tensor-core kernel's extra operands
struct BwdWs {
  size_t part_off, dw_off, pk_off, total;
};
inline BwdWs bwd_ws_layout(int B, int M, int d, int r) {
  BwdWs w;
  const int c1 = bwd_plan(B, M).chunks, c2 = bwd_tile_plan(B, M).chunks;
  const int chunks = c1 > c2 ? c1 : c2;
  w.part_off = align_up(attn_ws_bytes(B, d, r), 256);
  w.dw_off = w.part_off + align_up((size_t)B * chunks * 2 * d * kTokenSlots * sizeof(float), 256);
  w.pk_off = w.dw_off + align_up((size_t)B * 3 * d * d * sizeof(float), 256);
  w.total = w.pk_off + align_up((size_t)B * 4 * kTokenSlots * d * sizeof(__nv_bfloat16), 256);
  return w;
}

// ---- launchers (one per kernel file) --------------------------------------
cudaError_t launch_gram_simt(int B, int N, int d, solar_dtype_t dt, const void* H, float* gpart,
                             int* status, const GramPlan& plan, cudaStream_t st);
bool gram_umma_supported(int N, int d, solar_dtype_t dt);
cudaError_t launch_gram_umma(int B, int N, int d, const void* H, float* gpart, int* status,
                             const GramPlan& plan, cudaStream_t st);
// parts: partial Gram matrices per user; splits: status words per user
cudaError_t launch_eig(int B, int d, int r, solar_dtype_t dt, int route, int sweep_cap, int force_iters,
                       const float* gpart, const int* gram_status, int parts, int splits, float* gsum, float* S,
                       float* V, int* info, int* route_taken, cudaStream_t st);
// The eigensolver CTA of a user may end with that user's factor-token projections (Eq. 11):
// weights in the storage type, the attention workspace of all users.
struct EigFuse {
  const void* Wq; const void* Wk; const void* Wv;
  float scale;
  char* attn_ws;
};
cudaError_t launch_eig_tridiag(int B, int d, int r, solar_dtype_t dt, int route, int sweep_cap,
                               const float* gpart, const int* gram_status, int parts, int splits, float* gsum,
                               float* S, float* V, int* info, int* route_taken, const EigFuse* fuse,
                               cudaStream_t st);
int eig_subspace_dim(int d, int r);
cudaError_t launch_project_us(int B, int N, int d, int r, solar_dtype_t dt, const void* H,
                              const float* V, void* US, cudaStream_t st);
cudaError_t launch_svd_grad(int B, int d, int r, const float* S, const float* V, const float* dS,
                            const float* dV, float eps_rel, float* K, cudaStream_t st);
cudaError_t launch_attn_bwd(int B, int M, int d, int r, solar_dtype_t dt, const void* C, const void* dO,
                            const float* S, const float* V, const void* Wq, const void* Wk, const void* Wv,
                            float scale, unsigned flags, void* dC, float* dWq, float* dWk, float* dWv,
                            float* dS, float* dV, char* ws, const AttnWs& lay, const BwdWs& bl,
                            cudaStream_t st);
bool attn_bwd_umma_supported(int M, int d, solar_dtype_t dt);
cudaError_t launch_attn_bwd_umma(int B, int M, int d, int r, const void* C, const void* dO, unsigned flags,
                                 void* dC, float* part, void* pk, int tiles_per_cta, int chunks, const char* ws,
                                 const AttnWs& lay, cudaStream_t st);
bool project_us_umma_supported(int N, int d, int r, solar_dtype_t dt);
cudaError_t launch_project_us_umma(int B, int N, int d, int r, const void* H, const float* V, void* US,
                                   cudaStream_t st);
cudaError_t launch_attn_prepare(int B, int d, int r, solar_dtype_t dt, const float* S,
                                const float* V, const void* Wq, const void* Wk, const void* Wv,
                                float scale, char* ws, const AttnWs& lay, cudaStream_t st);
cudaError_t launch_attn_simt(int B, int M, int d, int r, solar_dtype_t dt, const void* C,
                             unsigned flags, void* O, const char* ws, const AttnWs& lay,
                             cudaStream_t st);
bool flash_factored_supported(int d, int r, solar_dtype_t dt);
cudaError_t launch_flash_factored(int B, int M, int N, int d, int r, const void* C, const void* US, void* O,
                                  const char* ws, const AttnWs& lay, cudaStream_t st);
bool attn_umma_supported(int d, solar_dtype_t dt);
// Throughput form of the tensor-core attention kernel: long CTAs that overlap the candidate
// stream, the GEMMs and the softmax of consecutive tiles (chosen under a slice limit).
bool attn_pipe_supported(int M, int d, int r, solar_dtype_t dt);
cudaError_t launch_attn_pipe(int B, int M, int r, const void* C, unsigned flags, void* O, const char* ws,
                             const AttnWs& lay, bool early_c, cudaStream_t st);
cudaError_t launch_attn_umma(int B, int M, int d, int r, const void* C, unsigned flags, void* O,
                             const char* ws, const AttnWs& lay, bool early_c, cudaStream_t st);

// ---- per-kernel launch limits -----------------------------------------------------------------
// Raises a kernel's dynamic shared-memory limit and asks for the largest shared-memory carve-out
// (an SM keeps ONE carve-out at a time: kernels of several requests share an SM only if they
// agree on it, and none of these kernels lives on L1), once per kernel and device: `done` is
// the call site's own table.  A lost race between host threads only repeats the two calls.
constexpr int kMaxDevicesCached = 64;
inline cudaError_t set_kernel_limits(const void* func, size_t smem_bytes, bool (&done)[kMaxDevicesCached]) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool cached = dev >= 0 && dev < kMaxDevicesCached;
  if (cached && done[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(func, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  if (cached) done[dev] = true;
  return cudaSuccess;
}

// ---- programmatic dependent launch ---------------------------------------------------
// The four kernels of a forward pass run back to back on one stream.  Launched with this
// attribute, a kernel may start while its predecessor is still draining; it does whatever
// does not depend on the predecessor (barrier set-up, staging weights, streaming H or the
// candidate tile) and then calls pdl_wait(), which returns once the predecessor has
// completed and its writes are visible.  pdl_trigger() lets the successor start launching; it
// is called late, when only a short tail is left, because CTAs that were launched early sit
// on shared memory and registers while they wait and would crowd out concurrent streams.
// Without the attribute both device calls are no-ops.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- device helpers ----------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// Loads 16 bytes of storage-type elements and widens them to fp32.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int kElems = 4;
  static __device__ __forceinline__ void load(const float* p, float* out) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* out) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

}  // namespace solar
