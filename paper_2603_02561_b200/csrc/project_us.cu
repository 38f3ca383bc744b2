// Right-multiplication of every history by a per-user matrix, Out_b = H_b X_b with X_b
// [d][q] fp32 and Out [B,N,q] in the storage type: the optional left factor
// US = U Sigma = H V (q = r; Eq. 10 eliminates U from the forward pass) and the backward
// pass of the SVD, dH = H K (q = d; Eq. 15).  This file holds the FFMA kernel for the shapes
// the tensor-core kernel does not take (fp32 storage, d = 32, N < 128).
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kRows = 64;
constexpr int kWarps = 8;
constexpr int kRP = 64;

template <typename T, int D>
__global__ void __launch_bounds__(kWarps * 32)
project_us_kernel(const T* __restrict__ H, const float* __restrict__ V, T* __restrict__ US, int N,
                  int r) {
  extern __shared__ float sm[];
  float* Vs = sm;                  // [D][kRP], zero padded
  float* Hs = sm + D * kRP;        // [kRows][D]
  const int b = blockIdx.y, n0 = blockIdx.x * kRows;
  const int c0 = blockIdx.z * kRP;       // this CTA's 64 output columns
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < D * kRP; e += kWarps * 32) {
    const int k = e / kRP, i = c0 + e % kRP;
    Vs[e] = i < r ? V[((size_t)b * D + k) * r + i] : 0.f;
  }
  constexpr int VE = Vec16<T>::kElems;
  constexpr int VPR = D / VE;
  const int rows = min(kRows, N - n0);
  const T* Hb = H + ((size_t)b * N + n0) * D;
  for (int v = tid; v < rows * VPR; v += kWarps * 32) {
    const int rr = v / VPR, cc = (v % VPR) * VE;
    float tmp[VE];
    Vec16<T>::load(Hb + (size_t)rr * D + cc, tmp);
#pragma unroll
    for (int e = 0; e < VE; ++e) Hs[rr * D + cc + e] = tmp[e];
  }
  __syncthreads();
  for (int rr = warp; rr < rows; rr += kWarps) {
    const float* h = Hs + rr * D;
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
    for (int k = 0; k < D; ++k) {
      s0 = fmaf(h[k], Vs[k * kRP + lane], s0);
      s1 = fmaf(h[k], Vs[k * kRP + lane + 32], s1);
    }
    T* o = US + ((size_t)b * N + n0 + rr) * r + c0;
    if (c0 + lane < r) o[lane] = from_f32<T>(s0);
    if (c0 + lane + 32 < r) o[lane + 32] = from_f32<T>(s1);
  }
}

template <typename T>
cudaError_t launch_t(int B, int N, int d, int r, const void* H, const float* V, void* US,
                     cudaStream_t st) {
  const dim3 grid((N + kRows - 1) / kRows, B, (r + kRP - 1) / kRP), block(kWarps * 32);
  const size_t smem = (size_t)(d * kRP + kRows * d) * sizeof(float);
  const T* h = static_cast<const T*>(H);
  T* u = static_cast<T*>(US);
#define SOLAR_US(DD)                                                                        \
  {                                                                                         \
    cudaError_t e = cudaFuncSetAttribute(project_us_kernel<T, DD>,                          \
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                         \
    project_us_kernel<T, DD><<<grid, block, smem, st>>>(h, V, u, N, r);                     \
  }
  switch (d) {
    case 32: SOLAR_US(32) break;
    case 64: SOLAR_US(64) break;
    case 128: SOLAR_US(128) break;
    default: return cudaErrorInvalidValue;
  }
#undef SOLAR_US
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_project_us(int B, int N, int d, int r, solar_dtype_t dt, const void* H,
                              const float* V, void* US, cudaStream_t st) {
  if (project_us_umma_supported(N, d, r, dt)) return launch_project_us_umma(B, N, d, r, H, V, US, st);
  return dt == SOLAR_BF16 ? launch_t<__nv_bfloat16>(B, N, d, r, H, V, US, st)
                          : launch_t<float>(B, N, d, r, H, V, US, st);
}

}  // namespace solar
