// SVD-Attention over the r factor tokens (Eq. 12), FFMA version.
// One warp per candidate row: scores = c T_b (lanes over tokens), softmax over
// the r tokens by warp shuffles, output = p Value_r (lanes over columns).
// Used for fp32 storage and for shapes the tensor-core kernel does not take.
#include <math.h>

#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kRows = 64;      // candidate rows per CTA
constexpr int kWarps = 8;
constexpr int kRP = 64;        // token slots (r <= 64), zero padded

template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32)
attn_simt_kernel(const T* __restrict__ C, T* __restrict__ O, const char* __restrict__ ws,
                 AttnWs lay, int M, int r, unsigned flags) {
  extern __shared__ float sm[];
  float* Ts = sm;                       // [D][kRP]
  float* Vs = Ts + D * kRP;             // [kRP][D]
  float* Cs = Vs + kRP * D;             // [kRows][D]
  float* Ps = Cs + kRows * D;           // [kWarps][kRP]

  const int b = blockIdx.y, m0 = blockIdx.x * kRows;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const char* wsb = ws + (size_t)b * lay.per_user;
  const float* Tf = reinterpret_cast<const float*>(wsb + lay.tf_off);
  const float* Vr = reinterpret_cast<const float*>(wsb + lay.vr_off);

  for (int e = tid; e < D * kRP; e += kWarps * 32) {
    const int k = e / kRP, i = e % kRP;
    Ts[e] = i < r ? Tf[k * r + i] : 0.f;
  }
  for (int e = tid; e < kRP * D; e += kWarps * 32) Vs[e] = e < r * D ? Vr[e] : 0.f;

  constexpr int VE = Vec16<T>::kElems;
  constexpr int VPR = D / VE;
  const T* Cb = C + ((size_t)b * M + m0) * D;
  const int rows = min(kRows, M - m0);
  for (int v = tid; v < kRows * VPR; v += kWarps * 32) {
    const int rr = v / VPR, cc = (v % VPR) * VE;
    float tmp[VE];
    if (rr < rows) {
      Vec16<T>::load(Cb + (size_t)rr * D + cc, tmp);
    } else {
#pragma unroll
      for (int e = 0; e < VE; ++e) tmp[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < VE; ++e) Cs[rr * D + cc + e] = tmp[e];
  }
  __syncthreads();

  const bool use_softmax = !(flags & SOLAR_FLAG_NO_SOFTMAX);
  float* P = Ps + warp * kRP;
  for (int rr = warp; rr < rows; rr += kWarps) {
    const float* c = Cs + rr * D;
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
    for (int k = 0; k < D; ++k) {
      const float ck = c[k];
      s0 = fmaf(ck, Ts[k * kRP + lane], s0);
      s1 = fmaf(ck, Ts[k * kRP + lane + 32], s1);
    }
    float p0, p1;
    if (use_softmax) {
      const float neg_inf = -INFINITY;
      const float a0 = lane < r ? s0 : neg_inf, a1 = lane + 32 < r ? s1 : neg_inf;
      float mx = fmaxf(a0, a1);
#pragma unroll
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float e0 = lane < r ? expf(a0 - mx) : 0.f;
      const float e1 = lane + 32 < r ? expf(a1 - mx) : 0.f;
      float sum = e0 + e1;
#pragma unroll
      for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      const float inv = 1.f / sum;
      p0 = e0 * inv; p1 = e1 * inv;
    } else {
      p0 = s0; p1 = s1;      // padded tokens have zero scores and zero Value_r rows
    }
    P[lane] = p0; P[lane + 32] = p1;
    __syncwarp();
    float out[D / 32];
#pragma unroll
    for (int jj = 0; jj < D / 32; ++jj) out[jj] = 0.f;
    for (int i = 0; i < r; ++i) {
      const float p = P[i];
#pragma unroll
      for (int jj = 0; jj < D / 32; ++jj) out[jj] = fmaf(p, Vs[i * D + lane + 32 * jj], out[jj]);
    }
    T* o = O + ((size_t)b * M + m0 + rr) * D;
#pragma unroll
    for (int jj = 0; jj < D / 32; ++jj) o[lane + 32 * jj] = from_f32<T>(out[jj]);
    __syncwarp();
  }
}

template <typename T>
cudaError_t launch_t(int B, int M, int d, int r, const void* C, unsigned flags, void* O,
                     const char* ws, const AttnWs& lay, cudaStream_t st) {
  const dim3 grid((M + kRows - 1) / kRows, B), block(kWarps * 32);
  const size_t smem = (size_t)(d * kRP + kRP * d + kRows * d + kWarps * kRP) * sizeof(float);
  const T* c = static_cast<const T*>(C);
  T* o = static_cast<T*>(O);
#define SOLAR_ATTN(DD)                                                                        \
  {                                                                                           \
    cudaError_t e = cudaFuncSetAttribute(attn_simt_kernel<T, DD>,                             \
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                           \
    attn_simt_kernel<T, DD><<<grid, block, smem, st>>>(c, o, ws, lay, M, r, flags);           \
  }
  switch (d) {
    case 32: SOLAR_ATTN(32) break;
    case 64: SOLAR_ATTN(64) break;
    case 128: SOLAR_ATTN(128) break;
    default: return cudaErrorInvalidValue;
  }
#undef SOLAR_ATTN
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_simt(int B, int M, int d, int r, solar_dtype_t dt, const void* C,
                             unsigned flags, void* O, const char* ws, const AttnWs& lay,
                             cudaStream_t st) {
  return dt == SOLAR_BF16 ? launch_t<__nv_bfloat16>(B, M, d, r, C, flags, O, ws, lay, st)
                          : launch_t<float>(B, M, d, r, C, flags, O, ws, lay, st);
}

}  // namespace solar
