// Per-user factor-token projections (Eq. 11):
//   Key_r   = (V Sigma)^T W_K   [r,d]
//   Value_r = (V Sigma)^T W_V   [r,d]
// and the folded score operand T_b = scale * W_Q Key_r^T [d,r], so that the
// scores of Eq. 12 are  scale * (C W_Q) Key_r^T = C T_b.
// Written to the workspace in fp32 and as bf16 operand images for the
// tensor-core attention kernel (T^T split into a high and a low bf16 half so
// that the score GEMM keeps ~16 mantissa bits; Value_r^T).
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kPrepThreads = 512;

template <typename T, int D>
__global__ void __launch_bounds__(kPrepThreads)
attn_prepare_kernel(const float* __restrict__ S, const float* __restrict__ V,
                    const T* __restrict__ Wq, const T* __restrict__ Wk, const T* __restrict__ Wv,
                    float scale, int r, char* __restrict__ ws, AttnWs lay) {
  extern __shared__ float sm[];
  float* VS = sm;            // [D][r]   V Sigma
  float* KrT = sm + D * r;   // [D][r]   Key_r^T
  const int b = blockIdx.x, tid = threadIdx.x;
  char* wsb = ws + (size_t)b * lay.per_user;
  float* Tf = reinterpret_cast<float*>(wsb + lay.tf_off);
  float* Vr = reinterpret_cast<float*>(wsb + lay.vr_off);
  __nv_bfloat16* Thi = reinterpret_cast<__nv_bfloat16*>(wsb + lay.thi_off);
  __nv_bfloat16* Tlo = reinterpret_cast<__nv_bfloat16*>(wsb + lay.tlo_off);
  __nv_bfloat16* VrT = reinterpret_cast<__nv_bfloat16*>(wsb + lay.vrt_off);

  for (int e = tid; e < D * r; e += kPrepThreads)
    VS[e] = V[(size_t)b * D * r + e] * S[(size_t)b * r + (e % r)];
  __syncthreads();

  // Key_r[i][j] = sum_k VS[k][i] Wk[k][j];  Value_r likewise with Wv.
  for (int e = tid; e < D * r; e += kPrepThreads) {
    const int i = e / D, j = e % D;          // j fastest: coalesced weight reads
    float ak = 0.f, av = 0.f;
#pragma unroll 8
    for (int k = 0; k < D; ++k) {
      const float vs = VS[k * r + i];
      ak = fmaf(vs, to_f32<T>(Wk[k * D + j]), ak);
      av = fmaf(vs, to_f32<T>(Wv[k * D + j]), av);
    }
    KrT[j * r + i] = ak;
    Vr[i * D + j] = av;
    VrT[j * r + i] = __float2bfloat16_rn(av);
  }
  __syncthreads();

  // T[k][i] = scale * sum_j Wq[k][j] Key_r[i][j]
  for (int e = tid; e < D * r; e += kPrepThreads) {
    const int k = e / r, i = e % r;          // i fastest: conflict-free KrT reads
    float acc = 0.f;
#pragma unroll 8
    for (int j = 0; j < D; ++j) acc = fmaf(to_f32<T>(Wq[k * D + j]), KrT[j * r + i], acc);
    acc *= scale;
    Tf[k * r + i] = acc;
    const __nv_bfloat16 hi = __float2bfloat16_rn(acc);
    Thi[i * D + k] = hi;
    Tlo[i * D + k] = __float2bfloat16_rn(acc - __bfloat162float(hi));
  }
}

template <typename T>
cudaError_t launch_t(int B, int d, int r, const float* S, const float* V, const void* Wq,
                     const void* Wk, const void* Wv, float scale, char* ws, const AttnWs& lay,
                     cudaStream_t st) {
  const size_t smem = (size_t)2 * d * r * sizeof(float);
  const T* q = static_cast<const T*>(Wq);
  const T* k = static_cast<const T*>(Wk);
  const T* v = static_cast<const T*>(Wv);
#define SOLAR_PREP(DD)                                                                          \
  {                                                                                             \
    cudaError_t e = cudaFuncSetAttribute(attn_prepare_kernel<T, DD>,                            \
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                             \
    attn_prepare_kernel<T, DD><<<B, kPrepThreads, smem, st>>>(S, V, q, k, v, scale, r, ws, lay); \
  }
  switch (d) {
    case 32: SOLAR_PREP(32) break;
    case 64: SOLAR_PREP(64) break;
    case 128: SOLAR_PREP(128) break;
    default: return cudaErrorInvalidValue;
  }
#undef SOLAR_PREP
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_prepare(int B, int d, int r, solar_dtype_t dt, const float* S,
                                const float* V, const void* Wq, const void* Wk, const void* Wv,
                                float scale, char* ws, const AttnWs& lay, cudaStream_t st) {
  return dt == SOLAR_BF16
             ? launch_t<__nv_bfloat16>(B, d, r, S, V, Wq, Wk, Wv, scale, ws, lay, st)
             : launch_t<float>(B, d, r, S, V, Wq, Wk, Wv, scale, ws, lay, st);
}

}  // namespace solar
