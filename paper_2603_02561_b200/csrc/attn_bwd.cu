// Backward pass of SVD-Attention through Eq. 11-12 (the chain rule of the forward
// definition; the paper prints no formulas for this part).  With the forward pass written
// as  S = C T,  T = scale W_Q Key_r^T,  P = softmax_r(S),  O = P Value_r:
//   dP = dO Value_r^T,  dS = P o (dP - rowsum(P o dP))      (dS = dP without the softmax)
//   dC = dS T^T,        dT = C^T dS,        dValue_r = P^T dO          (reductions over M)
//   dW_Q = scale dT Key_r,   dKey_r = scale dT^T W_Q,
//   dA = dKey_r W_K^T + dValue_r W_V^T,   A = Sigma V^T,
//   dW_K = A^T dKey_r,   dW_V = A^T dValue_r,   dSigma_i = sum_k dA_ik V_ki,   dV_ki = dA_ik sigma_i.
// Three kernels: the streaming one (one CTA per chunk of candidate rows; recomputes S and P,
// writes dC and a partial of dT and dValue_r^T), a per-user one (sums the partials in chunk
// order, runs the small chain, writes dSigma, dV and this user's dW contributions) and a
// sum over users in user order.  FFMA arithmetic in fp32 for every shape and storage type.
#include <math.h>

#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kBatch = 32;            // candidate rows per inner batch
constexpr int kRP = kTokenSlots;      // 64 token slots, zero padded

template <typename T> __device__ __forceinline__ T from_f32_(float x);
template <> __device__ __forceinline__ float from_f32_<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32_<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_bwd_rows_kernel(const T* __restrict__ C, const T* __restrict__ dO, T* __restrict__ dC,
                     const char* __restrict__ ws, AttnWs lay, float* __restrict__ part, int M, int r,
                     int rows_per_cta, unsigned flags) {
  constexpr int LT = kRP + 1;           // odd pitch: rows of T are read along k as well as along i
  constexpr int Q = D * kRP / kThreads; // accumulator entries per thread
  extern __shared__ __align__(16) float sm[];
  float* Ts = sm;                       // [D][LT]    T[k][i]
  float* VrT = Ts + D * LT;             // [D][kRP]   Value_r^T[j][i]
  float* Cs = VrT + D * kRP;            // [kBatch][D]
  float* Gs = Cs + kBatch * D;          // [kBatch][D]  dO rows
  float* Ps = Gs + kBatch * D;          // [kBatch][kRP]
  float* Ds = Ps + kBatch * kRP;        // [kBatch][kRP]  dS rows

  const int b = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const char* wsb = ws + (size_t)b * lay.per_user;
  const float* Tf = reinterpret_cast<const float*>(wsb + lay.tf_off);
  const float* Vr = reinterpret_cast<const float*>(wsb + lay.vr_off);
  for (int e = tid; e < D * kRP; e += kThreads) {
    const int k = e / kRP, i = e % kRP;
    Ts[k * LT + i] = i < r ? Tf[k * r + i] : 0.f;
    VrT[e] = i < r ? Vr[i * D + k] : 0.f;
  }
  const bool use_softmax = !(flags & SOLAR_FLAG_NO_SOFTMAX);
  float accT[Q], accV[Q];
#pragma unroll
  for (int q = 0; q < Q; ++q) { accT[q] = 0.f; accV[q] = 0.f; }

  constexpr int VE = Vec16<T>::kElems;
  constexpr int VPR = D / VE;
  const int m_begin = chunk * rows_per_cta;
  const int m_end = min(M, m_begin + rows_per_cta);
  for (int m0 = m_begin; m0 < m_end; m0 += kBatch) {
    __syncthreads();                    // the previous batch's buffers are free (and T, Value_r^T are staged)
    const int rows = min(kBatch, m_end - m0);
    for (int v = tid; v < kBatch * VPR; v += kThreads) {
      const int rr = v / VPR, cc = (v % VPR) * VE;
      float c[VE], g[VE];
      if (rr < rows) {
        Vec16<T>::load(C + ((size_t)b * M + m0 + rr) * D + cc, c);
        Vec16<T>::load(dO + ((size_t)b * M + m0 + rr) * D + cc, g);
      } else {
#pragma unroll
        for (int e = 0; e < VE; ++e) { c[e] = 0.f; g[e] = 0.f; }
      }
#pragma unroll
      for (int e = 0; e < VE; ++e) { Cs[rr * D + cc + e] = c[e]; Gs[rr * D + cc + e] = g[e]; }
    }
    __syncthreads();

    // scores, probabilities and dS of four rows per warp; lanes run over the tokens
    for (int rr = warp; rr < kBatch; rr += kWarps) {
      const float* c = Cs + rr * D;
      const float* g = Gs + rr * D;
      float s0 = 0.f, s1 = 0.f, d0 = 0.f, d1 = 0.f;
#pragma unroll 8
      for (int k = 0; k < D; ++k) {
        const float ck = c[k], gk = g[k];
        s0 = fmaf(ck, Ts[k * LT + lane], s0);
        s1 = fmaf(ck, Ts[k * LT + lane + 32], s1);
        d0 = fmaf(gk, VrT[k * kRP + lane], d0);
        d1 = fmaf(gk, VrT[k * kRP + lane + 32], d1);
      }
      float p0, p1, ds0, ds1;
      if (use_softmax) {
        const float a0 = lane < r ? s0 : -INFINITY, a1 = lane + 32 < r ? s1 : -INFINITY;
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
        float dot = fmaf(p0, d0, p1 * d1);
#pragma unroll
        for (int o = 16; o; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
        ds0 = p0 * (d0 - dot); ds1 = p1 * (d1 - dot);
      } else {
        p0 = lane < r ? s0 : 0.f; p1 = lane + 32 < r ? s1 : 0.f;
        ds0 = lane < r ? d0 : 0.f; ds1 = lane + 32 < r ? d1 : 0.f;
      }
      const bool live = rr < rows;       // rows past the end contribute nothing
      Ps[rr * kRP + lane] = live ? p0 : 0.f;  Ps[rr * kRP + lane + 32] = live ? p1 : 0.f;
      Ds[rr * kRP + lane] = live ? ds0 : 0.f; Ds[rr * kRP + lane + 32] = live ? ds1 : 0.f;
    }
    __syncthreads();

    // dC[m][k] = sum_i dS[m][i] T[k][i]; lanes run over k
    for (int e = tid; e < kBatch * D; e += kThreads) {
      const int rr = e / D, k = e % D;
      if (rr < rows) {
        float acc = 0.f;
#pragma unroll 8
        for (int i = 0; i < kRP; ++i) acc = fmaf(Ds[rr * kRP + i], Ts[k * LT + i], acc);
        dC[((size_t)b * M + m0 + rr) * D + k] = from_f32_<T>(acc);
      }
    }
    // dT[k][i] += sum_m C[m][k] dS[m][i],  dValue_r^T[k][i] += sum_m dO[m][k] P[m][i]
#pragma unroll
    for (int q = 0; q < Q; ++q) {
      const int e = tid + q * kThreads, k = e / kRP, i = e % kRP;
      float at = accT[q], av = accV[q];
#pragma unroll 8
      for (int m = 0; m < kBatch; ++m) {
        at = fmaf(Cs[m * D + k], Ds[m * kRP + i], at);
        av = fmaf(Gs[m * D + k], Ps[m * kRP + i], av);
      }
      accT[q] = at; accV[q] = av;
    }
  }
  float* out = part + ((size_t)b * gridDim.x + chunk) * 2 * D * kRP;
#pragma unroll
  for (int q = 0; q < Q; ++q) {
    const int e = tid + q * kThreads;
    out[e] = accT[q];
    out[D * kRP + e] = accV[q];
  }
}

// Per-user chain from dT and dValue_r to dSigma, dV and this user's dW contributions.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_bwd_user_kernel(const float* __restrict__ part, int chunks, const float* __restrict__ S,
                     const float* __restrict__ V, const T* __restrict__ Wq, const T* __restrict__ Wk,
                     const T* __restrict__ Wv, float scale, int r, float* __restrict__ dS,
                     float* __restrict__ dV, float* __restrict__ dw) {
  extern __shared__ __align__(16) float sm[];
  float* dT = sm;                       // [D][kRP]   dT[k][i]
  float* dVT = dT + D * kRP;            // [D][kRP]   dValue_r^T[j][i]
  float* A = dVT + D * kRP;             // [kRP][D]   Sigma V^T
  float* X = A + kRP * D;               // [kRP][D]   Key_r, then dKey_r
  float* dA = X + kRP * D;              // [kRP][D]
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // partials in chunk order
  for (int e = tid; e < 2 * D * kRP; e += kThreads) {
    float acc = 0.f;
    for (int c = 0; c < chunks; ++c) acc += part[((size_t)b * chunks + c) * 2 * D * kRP + e];
    dT[e] = acc;                        // dVT follows dT in shared memory
  }
  for (int e = tid; e < kRP * D; e += kThreads) {
    const int i = e / D, k = e % D;
    A[e] = i < r ? S[(size_t)b * r + i] * V[((size_t)b * D + k) * r + i] : 0.f;
  }
  __syncthreads();
  // Key_r[i][j] = sum_k A[i][k] W_K[k][j]; lanes run over j
  for (int e = tid; e < r * D; e += kThreads) {
    const int i = e / D, j = e % D;
    float acc = 0.f;
#pragma unroll 4
    for (int k = 0; k < D; ++k) acc = fmaf(A[i * D + k], to_f32<T>(Wk[k * D + j]), acc);
    X[e] = acc;
  }
  __syncthreads();
  float* dWq = dw + (size_t)b * 3 * D * D;
  float* dWk = dWq + D * D;
  float* dWv = dWk + D * D;
  // dW_Q[k][j] = scale sum_i dT[k][i] Key_r[i][j]
  for (int e = tid; e < D * D; e += kThreads) {
    const int k = e / D, j = e % D;
    float acc = 0.f;
    for (int i = 0; i < r; ++i) acc = fmaf(dT[k * kRP + i], X[i * D + j], acc);
    dWq[e] = scale * acc;
  }
  __syncthreads();
  // dKey_r[i][j] = scale sum_k dT[k][i] W_Q[k][j]   (over Key_r)
  for (int e = tid; e < r * D; e += kThreads) {
    const int i = e / D, j = e % D;
    float acc = 0.f;
#pragma unroll 4
    for (int k = 0; k < D; ++k) acc = fmaf(dT[k * kRP + i], to_f32<T>(Wq[k * D + j]), acc);
    X[e] = scale * acc;
  }
  __syncthreads();
  // dW_K[k][j] = sum_i A[i][k] dKey_r[i][j],  dW_V[k][j] = sum_i A[i][k] dValue_r[i][j]
  for (int e = tid; e < D * D; e += kThreads) {
    const int k = e / D, j = e % D;
    float ak = 0.f, av = 0.f;
    for (int i = 0; i < r; ++i) {
      const float a = A[i * D + k];
      ak = fmaf(a, X[i * D + j], ak);
      av = fmaf(a, dVT[j * kRP + i], av);
    }
    dWk[e] = ak;
    dWv[e] = av;
  }
  // dA[i][k] = sum_j dKey_r[i][j] W_K[k][j] + dValue_r[i][j] W_V[k][j]: one warp per entry,
  // lanes run over j (rows of the weights are read as they are stored)
  for (int e = warp; e < r * D; e += kWarps) {
    const int i = e / D, k = e % D;
    float acc = 0.f;
    for (int j = lane; j < D; j += 32)
      acc = fmaf(X[i * D + j], to_f32<T>(Wk[k * D + j]), fmaf(dVT[j * kRP + i], to_f32<T>(Wv[k * D + j]), acc));
#pragma unroll
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) dA[e] = acc;
  }
  __syncthreads();
  // dSigma_i = sum_k dA[i][k] V[k][i],  dV[k][i] = dA[i][k] sigma_i
  for (int i = warp; i < r; i += kWarps) {
    float acc = 0.f;
    for (int k = lane; k < D; k += 32) acc = fmaf(dA[i * D + k], V[((size_t)b * D + k) * r + i], acc);
#pragma unroll
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) dS[(size_t)b * r + i] = acc;
  }
  for (int e = tid; e < D * r; e += kThreads) {
    const int k = e / r, i = e % r;
    dV[(size_t)b * D * r + e] = dA[i * D + k] * S[(size_t)b * r + i];
  }
}

// out[w][e] = sum over users (in user order) of dw[b][w][e]
__global__ void sum_users_kernel(const float* __restrict__ dw, int B, int n, float* __restrict__ o0,
                                 float* __restrict__ o1, float* __restrict__ o2) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  const int w = blockIdx.y;
  if (e >= n) return;
  float acc = 0.f;
  for (int b = 0; b < B; ++b) acc += dw[((size_t)b * 3 + w) * n + e];
  (w == 0 ? o0 : w == 1 ? o1 : o2)[e] = acc;
}

template <typename T, int D>
cudaError_t launch_td(int B, int M, int r, const void* C, const void* dO, const float* S, const float* V,
                      const void* Wq, const void* Wk, const void* Wv, float scale, unsigned flags, void* dC,
                      float* dWq, float* dWk, float* dWv, float* dS, float* dV, char* ws, const AttnWs& lay,
                      const BwdWs& bl, cudaStream_t st) {
  const BwdPlan plan = bwd_plan(B, M);
  float* part = reinterpret_cast<float*>(ws + bl.part_off);
  float* dw = reinterpret_cast<float*>(ws + bl.dw_off);
  const size_t smem_rows = (size_t)(D * (kRP + 1) + D * kRP + 2 * kBatch * D + 2 * kBatch * kRP) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(attn_bwd_rows_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem_rows);
  if (e != cudaSuccess) return e;
  attn_bwd_rows_kernel<T, D><<<dim3(plan.chunks, B), kThreads, smem_rows, st>>>(
      static_cast<const T*>(C), static_cast<const T*>(dO), static_cast<T*>(dC), ws, lay, part, M, r,
      plan.rows_per_cta, flags);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem_user = (size_t)(2 * D * kRP + 3 * kRP * D) * sizeof(float);
  e = cudaFuncSetAttribute(attn_bwd_user_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_user);
  if (e != cudaSuccess) return e;
  attn_bwd_user_kernel<T, D><<<B, kThreads, smem_user, st>>>(part, plan.chunks, S, V, static_cast<const T*>(Wq),
                                                            static_cast<const T*>(Wk), static_cast<const T*>(Wv),
                                                            scale, r, dS, dV, dw);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  sum_users_kernel<<<dim3((D * D + 255) / 256, 3), 256, 0, st>>>(dw, B, D * D, dWq, dWk, dWv);
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_t(int B, int M, int d, int r, const void* C, const void* dO, const float* S, const float* V,
                     const void* Wq, const void* Wk, const void* Wv, float scale, unsigned flags, void* dC,
                     float* dWq, float* dWk, float* dWv, float* dS, float* dV, char* ws, const AttnWs& lay,
                     const BwdWs& bl, cudaStream_t st) {
  switch (d) {
    case 32: return launch_td<T, 32>(B, M, r, C, dO, S, V, Wq, Wk, Wv, scale, flags, dC, dWq, dWk, dWv, dS, dV, ws, lay, bl, st);
    case 64: return launch_td<T, 64>(B, M, r, C, dO, S, V, Wq, Wk, Wv, scale, flags, dC, dWq, dWk, dWv, dS, dV, ws, lay, bl, st);
    case 128: return launch_td<T, 128>(B, M, r, C, dO, S, V, Wq, Wk, Wv, scale, flags, dC, dWq, dWk, dWv, dS, dV, ws, lay, bl, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_attn_bwd(int B, int M, int d, int r, solar_dtype_t dt, const void* C, const void* dO,
                            const float* S, const float* V, const void* Wq, const void* Wk, const void* Wv,
                            float scale, unsigned flags, void* dC, float* dWq, float* dWk, float* dWv,
                            float* dS, float* dV, char* ws, const AttnWs& lay, const BwdWs& bl,
                            cudaStream_t st) {
  return dt == SOLAR_BF16
             ? launch_t<__nv_bfloat16>(B, M, d, r, C, dO, S, V, Wq, Wk, Wv, scale, flags, dC, dWq, dWk, dWv, dS, dV, ws, lay, bl, st)
             : launch_t<float>(B, M, d, r, C, dO, S, V, Wq, Wk, Wv, scale, flags, dC, dWq, dWk, dWv, dS, dV, ws, lay, bl, st);
}

}  // namespace solar
