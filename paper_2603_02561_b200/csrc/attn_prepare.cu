// Per-user factor-token projections (Eq. 11):
//   Key_r   = (V Sigma)^T W_K   [r,d]
//   Value_r = (V Sigma)^T W_V   [r,d]
// and the folded score operand T_b = scale * W_Q Key_r^T [d,r], so that the
// scores of Eq. 12 are  scale * (C W_Q) Key_r^T = C T_b.
// Written to the workspace in fp32 (for the FFMA attention kernel) and as packed bf16
// operand images for the tensor-core attention kernel: T^T and Value_r^T, each split
// into a high and a low bf16 half so that both GEMMs keep ~16 mantissa bits, zero padded
// to 64 token slots.
//
// Two CTAs per user: one computes Key_r^T and T (W_K, W_Q), the other Value_r (W_V).
// Each weight matrix is staged once in shared memory with coalesced 16-byte loads; the small
// products then run out of shared memory with 4 outputs per thread.
#include "project_mma.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kPrepThreads = 512;

// Stages W[D][D] (storage type T) as fp32 in shared memory.
template <typename T, int D>
__device__ __forceinline__ void stage_weight(const T* __restrict__ W, float* __restrict__ Ws, int tid) {
  constexpr int VE = Vec16<T>::kElems;
  for (int v = tid; v < D * D / VE; v += kPrepThreads) {
    float tmp[VE];
    Vec16<T>::load(W + (size_t)v * VE, tmp);
#pragma unroll
    for (int e = 0; e < VE; ++e) Ws[v * VE + e] = tmp[e];
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kPrepThreads)
attn_prepare_kernel(const float* __restrict__ S, const float* __restrict__ V,
                    const T* __restrict__ Wq, const T* __restrict__ Wk, const T* __restrict__ Wv,
                    float scale, int r, char* __restrict__ ws, AttnWs lay) {
  extern __shared__ __align__(16) float sm[];
  const int rp = (r + 3) & ~3;          // token pitch: rows of VS / KrT are read 4 at a time
  float* Ws = sm;                       // [D][D]   W_K (role 0) or W_V (role 1)
  float* Wq_s = Ws + D * D;             // [D][D]   W_Q (role 0)
  float* VS = Wq_s + D * D;             // [D][rp]  V Sigma (zero in the padding)
  float* KrT = VS + D * rp;             // [D][rp]  Key_r^T
  const int b = blockIdx.x, role = blockIdx.y, tid = threadIdx.x;
  char* wsb = ws + (size_t)b * lay.per_user;
  float* Tf = reinterpret_cast<float*>(wsb + lay.tf_off);
  float* Vr = reinterpret_cast<float*>(wsb + lay.vr_off);
  __nv_bfloat16* Tpk = reinterpret_cast<__nv_bfloat16*>(wsb + lay.tpk_off);
  __nv_bfloat16* Vpk = reinterpret_cast<__nv_bfloat16*>(wsb + lay.vpk_off);
  const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);

  // S and V come from the eigensolver, the weights from the caller (a kernel earlier on the
  // stream may have written them), and the workspace may still be in use: nothing is read or
  // written before the previous kernel has completed
  pdl_wait();
  stage_weight<T, D>(role == 0 ? Wk : Wv, Ws, tid);
  if (role == 0) stage_weight<T, D>(Wq, Wq_s, tid);
  for (int e = tid; e < D * rp; e += kPrepThreads) {
    const int k = e / rp, i = e % rp;
    VS[e] = i < r ? V[((size_t)b * D + k) * r + i] * (S != nullptr ? S[(size_t)b * r + i] : 1.f) : 0.f;
  }
  // zero padding of the packed operands: token slots r .. 63
  if (role == 0) {
    for (int e = tid; e < 2 * (kTokenSlots - r) * D; e += kPrepThreads) {
      const int h = e / ((kTokenSlots - r) * D), rem = e % ((kTokenSlots - r) * D);
      Tpk[((size_t)h * kTokenSlots + r) * D + rem] = zero;
    }
  } else {
    for (int e = tid; e < 2 * D * (kTokenSlots - r); e += kPrepThreads) {
      const int row = e / (kTokenSlots - r), i = r + e % (kTokenSlots - r);
      Vpk[(size_t)row * kTokenSlots + i] = zero;      // row runs over [2][D]
    }
  }
  __syncthreads();
  pdl_trigger();       // the next kernel may start launching while the products run

  // X[i][j] = sum_k VS[k][i] W[k][j] for four tokens i per thread; j runs along the lanes.
  auto project = [&](float (&acc)[4], int i0, int j) {
#pragma unroll
    for (int m = 0; m < 4; ++m) acc[m] = 0.f;
#pragma unroll 8
    for (int k = 0; k < D; ++k) {
      const float w = Ws[k * D + j];
      const float4 vs = *reinterpret_cast<const float4*>(VS + k * rp + i0);
      acc[0] = fmaf(vs.x, w, acc[0]); acc[1] = fmaf(vs.y, w, acc[1]);
      acc[2] = fmaf(vs.z, w, acc[2]); acc[3] = fmaf(vs.w, w, acc[3]);
    }
  };

  if (role == 1) {
    // Value_r (fp32) and Value_r^T (packed bf16 halves)
    for (int t = tid; t < (rp / 4) * D; t += kPrepThreads) {
      const int j = t % D, i0 = (t / D) * 4;
      float acc[4];
      project(acc, i0, j);
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const int i = i0 + m;
        if (i < r) {
          Vr[i * D + j] = acc[m];
          const __nv_bfloat16 hi = __float2bfloat16_rn(acc[m]);
          Vpk[(size_t)j * kTokenSlots + i] = hi;
          Vpk[(size_t)(D + j) * kTokenSlots + i] = __float2bfloat16_rn(acc[m] - __bfloat162float(hi));
        }
      }
    }
    return;
  }

  // Key_r^T
  for (int t = tid; t < (rp / 4) * D; t += kPrepThreads) {
    const int j = t % D, i0 = (t / D) * 4;
    float acc[4];
    project(acc, i0, j);
    *reinterpret_cast<float4*>(KrT + j * rp + i0) = make_float4(acc[0], acc[1], acc[2], acc[3]);
  }
  __syncthreads();
  // T[k][i] = scale * sum_j Wq[k][j] Key_r[i][j], four tokens i per thread
  for (int t = tid; t < (rp / 4) * D; t += kPrepThreads) {
    const int i0 = (t % (rp / 4)) * 4, k = t / (rp / 4);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
    for (int j = 0; j < D; ++j) {
      const float w = Wq_s[k * D + j];
      const float4 kr = *reinterpret_cast<const float4*>(KrT + j * rp + i0);
      acc[0] = fmaf(w, kr.x, acc[0]); acc[1] = fmaf(w, kr.y, acc[1]);
      acc[2] = fmaf(w, kr.z, acc[2]); acc[3] = fmaf(w, kr.w, acc[3]);
    }
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const int i = i0 + m;
      if (i < r) {
        const float v = acc[m] * scale;
        Tf[k * r + i] = v;
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        Tpk[(size_t)i * D + k] = hi;
        Tpk[((size_t)kTokenSlots + i) * D + k] = __float2bfloat16_rn(v - __bfloat162float(hi));
      }
    }
  }
}

// bf16 weights, d = 64 or 128: one CTA per user, the three products on the tensor cores (the
// routine the eigensolver's epilogue uses, so a forward pass gives the same bits either way).
template <int D>
__global__ void __launch_bounds__(D == 128 ? 256 : 128, 1)
attn_prepare_mma_kernel(const float* __restrict__ S, const float* __restrict__ V, const void* __restrict__ Wq,
                        const void* __restrict__ Wk, const void* __restrict__ Wv, float scale, int r,
                        char* __restrict__ ws, AttnWs lay) {
  constexpr int NT = D == 128 ? 256 : 128;
  extern __shared__ __align__(16) unsigned char smb[];
  const int rp = (r + 3) & ~3;
  const int b = blockIdx.x, tid = threadIdx.x;
  char* wsb = ws + (size_t)b * lay.per_user;
  float* VS = reinterpret_cast<float*>(smb);     // [D][rp]  V Sigma (zero in the padding)
  pdl_wait();                                    // as in the kernel above
  for (int e = tid; e < D * rp; e += NT) {
    const int k = e / rp, i = e % rp;
    VS[e] = i < r ? V[((size_t)b * D + k) * r + i] * (S != nullptr ? S[(size_t)b * r + i] : 1.f) : 0.f;
  }
  __syncthreads();
  pdl_trigger();
  pmma::project<D, NT>(smb, r, Wq, Wk, Wv, scale, reinterpret_cast<__nv_bfloat16*>(wsb + lay.tpk_off),
                       reinterpret_cast<__nv_bfloat16*>(wsb + lay.vpk_off), reinterpret_cast<float*>(wsb + lay.tf_off),
                       reinterpret_cast<float*>(wsb + lay.vr_off), kTokenSlots, tid);
}

template <int D>
cudaError_t launch_mma(int B, int r, const float* S, const float* V, const void* Wq, const void* Wk, const void* Wv,
                       float scale, char* ws, const AttnWs& lay, cudaStream_t st) {
  static bool limits_set[kMaxDevicesCached] = {};
  cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&attn_prepare_mma_kernel<D>),
                                    (size_t)pmma::Lay<D>::bytes(kTokenSlots), limits_set);
  if (e != cudaSuccess) return e;
  e = launch_pdl(attn_prepare_mma_kernel<D>, dim3(B), dim3(D == 128 ? 256 : 128),
                 (size_t)pmma::Lay<D>::bytes((r + 15) & ~15), st, S, V, Wq, Wk, Wv, scale, r, ws, lay);
  return e != cudaSuccess ? e : cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(int B, int d, int r, const float* S, const float* V, const void* Wq,
                     const void* Wk, const void* Wv, float scale, char* ws, const AttnWs& lay,
                     cudaStream_t st) {
  const int rp = (r + 3) & ~3;
  const size_t smem = (size_t)(2 * d * d + 2 * d * rp) * sizeof(float);
  const T* q = static_cast<const T*>(Wq);
  const T* k = static_cast<const T*>(Wk);
  const T* v = static_cast<const T*>(Wv);
#define SOLAR_PREP(DD)                                                                          \
  {                                                                                             \
    static bool limits_set[kMaxDevicesCached] = {};                                             \
    cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&attn_prepare_kernel<T, DD>), \
                                      (size_t)(2 * DD * DD + 2 * DD * 64) * sizeof(float), limits_set); \
    if (e != cudaSuccess) return e;                                                             \
    e = launch_pdl(attn_prepare_kernel<T, DD>, dim3(B, 2), dim3(kPrepThreads), smem, st, S, V, q, k, v, \
                   scale, r, ws, lay);                                                           \
    if (e != cudaSuccess) return e;                                                             \
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
  if (dt == SOLAR_BF16 && d == 64) return launch_mma<64>(B, r, S, V, Wq, Wk, Wv, scale, ws, lay, st);
  if (dt == SOLAR_BF16 && d == 128) return launch_mma<128>(B, r, S, V, Wq, Wk, Wv, scale, ws, lay, st);
  return dt == SOLAR_BF16
             ? launch_t<__nv_bfloat16>(B, d, r, S, V, Wq, Wk, Wv, scale, ws, lay, st)
             : launch_t<float>(B, d, r, S, V, Wq, Wk, Wv, scale, ws, lay, st);
}

}  // namespace solar
