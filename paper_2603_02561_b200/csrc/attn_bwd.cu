// Backward pass of SVD-Attention through Eq. 11-12 (the chain rule of the forward
// definition; the paper prints no formulas for this part).  With the forward pass written
// as  S = C T,  T = scale W_Q Key_r^T,  P = softmax_r(S),  O = P Value_r:
//   dP = dO Value_r^T,  dS = P o (dP - rowsum(P o dP))      (dS = dP without the softmax)
//   dC = dS T^T,        dT = C^T dS,        dValue_r = P^T dO          (reductions over M)
//   dW_Q = scale dT Key_r,   dKey_r = scale dT^T W_Q,
//   dA = dKey_r W_K^T + dValue_r W_V^T,   A = Sigma V^T,
//   dW_K = A^T dKey_r,   dW_V = A^T dValue_r,   dSigma_i = sum_k dA_ik V_ki,   dV_ki = dA_ik sigma_i.
// Four kernels: the streaming one (one CTA per chunk of candidate rows; recomputes S and P,
// writes dC and a partial of dT and dValue_r^T), the sum of the partials in chunk order, a
// per-user one (the small chain; writes dSigma, dV and this user's dW contributions) and a
// sum over users in user order.  The streaming kernel here is the FFMA one (fp32 storage,
// d = 32); bf16 storage with d = 64 or 128 takes the tensor-core kernel instead.
#include <math.h>

#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kUserThreads = 1024;   // the per-user chain is latency-bound: many warps per scheduler
constexpr int kUserWarps = kUserThreads / 32;
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

// out(m, n) = sum_k a(m, k) b(k, n) for m < rows (rounded up to 4), n < D, by the whole CTA:
// a warp takes four rows at a time, its lanes run along n with D/32 columns each, so one
// step of k costs 4 broadcast reads of a and D/32 reads of b for 4*D/32 FMAs (the plain
// one-output-per-thread loop is bound by shared-memory issue, not by the FMAs).
template <int D, typename FA, typename FB, typename FS>
__device__ __forceinline__ void small_gemm(int rows, int K, FA a, FB b, FS store, int warp, int lane,
                                           int nwarps) {
  constexpr int NC = D / 32;
  for (int m0 = warp * 4; m0 < rows; m0 += nwarps * 4) {
    float acc[4][NC];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int c = 0; c < NC; ++c) acc[x][c] = 0.f;
#pragma unroll 4
    for (int k = 0; k < K; ++k) {
      float av[4], bv[NC];
#pragma unroll
      for (int x = 0; x < 4; ++x) av[x] = a(m0 + x, k);
#pragma unroll
      for (int c = 0; c < NC; ++c) bv[c] = b(k, lane + 32 * c);
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[x][c] = fmaf(av[x], bv[c], acc[x][c]);
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int c = 0; c < NC; ++c)
        if (m0 + x < rows) store(m0 + x, lane + 32 * c, acc[x][c]);
  }
}

// Per-user chain from dT and dValue_r to dSigma, dV and this user's dW contributions.
// Each weight matrix is staged in shared memory (fp32, odd pitch) when it is needed: W_K for
// Key_r, W_Q for dKey_r, then W_K and W_V again for dA, where they are read along their rows.
template <typename T, int D>
__global__ void __launch_bounds__(kUserThreads)
attn_bwd_user_kernel(const float* __restrict__ part, int chunks, const float* __restrict__ S,
                     const float* __restrict__ V, const T* __restrict__ Wq, const T* __restrict__ Wk,
                     const T* __restrict__ Wv, float scale, int r, float* __restrict__ dS,
                     float* __restrict__ dV, float* __restrict__ dw) {
  extern __shared__ __align__(16) float sm[];
  constexpr int LR = kRP + 1;           // odd pitch: dT and dValue_r^T are read along both indices
  constexpr int LW = D + 1;             // odd pitch of the staged weight matrix
  float* dT = sm;                       // [D][LR]    dT[k][i]
  float* dVT = dT + D * LR;             // [D][LR]    dValue_r^T[j][i]
  float* A = dVT + D * LR;              // [kRP][D]   Sigma V^T (rows past r zero), at the end dA
  float* X = A + kRP * D;               // [kRP][D]   Key_r, then dKey_r (rows past r zero)
  float* Ws = X + kRP * D;              // [D][LW]    the weight matrix in use
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  auto stage = [&](const T* __restrict__ W) {
    constexpr int VE = Vec16<T>::kElems;
    for (int v = tid; v < D * D / VE; v += kUserThreads) {
      float tmp[VE];
      Vec16<T>::load(W + (size_t)v * VE, tmp);
      const int k = (v * VE) / D, j = (v * VE) % D;
#pragma unroll
      for (int e = 0; e < VE; ++e) Ws[k * LW + j + e] = tmp[e];
    }
  };

  stage(Wk);
  // the partials, summed into the first chunk's slot by sum_chunks_kernel
  for (int e = tid; e < 2 * D * kRP; e += kUserThreads)
    dT[(e / kRP) * LR + e % kRP] = part[(size_t)b * chunks * 2 * D * kRP + e];   // dVT follows dT in shared memory
  for (int e = tid; e < kRP * D; e += kUserThreads) {
    const int k = e / kRP, i = e % kRP;   // V is read along its rows
    A[i * D + k] = i < r ? S[(size_t)b * r + i] * V[((size_t)b * D + k) * r + i] : 0.f;
    X[e] = 0.f;
  }
  __syncthreads();
  // Key_r[i][j] = sum_k A[i][k] W_K[k][j]
  small_gemm<D>(r, D, [&](int i, int k) { return A[i * D + k]; }, [&](int k, int j) { return Ws[k * LW + j]; },
                [&](int i, int j, float v) { X[i * D + j] = v; }, warp, lane, kUserWarps);
  __syncthreads();
  stage(Wq);
  float* dWq = dw + (size_t)b * 3 * D * D;
  float* dWk = dWq + D * D;
  float* dWv = dWk + D * D;
  // dW_Q[k][j] = scale sum_i dT[k][i] Key_r[i][j]
  small_gemm<D>(D, r, [&](int k, int i) { return dT[k * LR + i]; }, [&](int i, int j) { return X[i * D + j]; },
                [&](int k, int j, float v) { dWq[k * D + j] = scale * v; }, warp, lane, kUserWarps);
  __syncthreads();
  // dKey_r[i][j] = scale sum_k dT[k][i] W_Q[k][j]   (over Key_r)
  small_gemm<D>(r, D, [&](int i, int k) { return dT[k * LR + i]; }, [&](int k, int j) { return Ws[k * LW + j]; },
                [&](int i, int j, float v) { X[i * D + j] = scale * v; }, warp, lane, kUserWarps);
  __syncthreads();
  stage(Wk);
  // dW_K[k][j] = sum_i A[i][k] dKey_r[i][j],  dW_V[k][j] = sum_i A[i][k] dValue_r[i][j]
  small_gemm<D>(D, r, [&](int k, int i) { return A[i * D + k]; }, [&](int i, int j) { return X[i * D + j]; },
                [&](int k, int j, float v) { dWk[k * D + j] = v; }, warp, lane, kUserWarps);
  small_gemm<D>(D, r, [&](int k, int i) { return A[i * D + k]; }, [&](int i, int j) { return dVT[j * LR + i]; },
                [&](int k, int j, float v) { dWv[k * D + j] = v; }, warp, lane, kUserWarps);
  __syncthreads();
  // dA[i][k] = sum_j dKey_r[i][j] W_K[k][j] + dValue_r[i][j] W_V[k][j]; dA takes the place of A
  small_gemm<D>(r, D, [&](int i, int j) { return X[i * D + j]; }, [&](int j, int k) { return Ws[k * LW + j]; },
                [&](int i, int k, float v) { A[i * D + k] = v; }, warp, lane, kUserWarps);
  __syncthreads();
  stage(Wv);
  __syncthreads();
  small_gemm<D>(r, D, [&](int i, int j) { return dVT[j * LR + i]; }, [&](int j, int k) { return Ws[k * LW + j]; },
                [&](int i, int k, float v) { A[i * D + k] += v; }, warp, lane, kUserWarps);
  __syncthreads();
  const float* dA = A;
  // dSigma_i = sum_k dA[i][k] V[k][i],  dV[k][i] = dA[i][k] sigma_i
  for (int i = warp; i < r; i += kUserWarps) {
    float acc = 0.f;
    for (int k = lane; k < D; k += 32) acc = fmaf(dA[i * D + k], V[((size_t)b * D + k) * r + i], acc);
#pragma unroll
    for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) dS[(size_t)b * r + i] = acc;
  }
  for (int e = tid; e < D * r; e += kUserThreads) {
    const int k = e / r, i = e % r;
    dV[(size_t)b * D * r + e] = dA[i * D + k] * S[(size_t)b * r + i];
  }
}

// part[b][0][e] = sum over the chunks (in chunk order) of part[b][c][e]
__global__ void sum_chunks_kernel(float* __restrict__ part, int chunks, int n) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= n) return;
  float* p = part + (size_t)blockIdx.y * chunks * n + e;
  float acc = 0.f;
  for (int c = 0; c < chunks; ++c) acc += p[(size_t)c * n];
  p[0] = acc;
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
  float* part = reinterpret_cast<float*>(ws + bl.part_off);
  float* dw = reinterpret_cast<float*>(ws + bl.dw_off);
  int chunks;
  cudaError_t e;
  if (attn_bwd_umma_supported(M, D, sizeof(T) == 2 ? SOLAR_BF16 : SOLAR_F32)) {
    const BwdTilePlan tp = bwd_tile_plan(B, M);
    chunks = tp.chunks;
    e = launch_attn_bwd_umma(B, M, D, r, C, dO, flags, dC, part, ws + bl.pk_off, tp.tiles_per_cta, tp.chunks, ws,
                             lay, st);
    if (e != cudaSuccess) return e;
  } else {
    const BwdPlan plan = bwd_plan(B, M);
    chunks = plan.chunks;
    const size_t smem_rows =
        (size_t)(D * (kRP + 1) + D * kRP + 2 * kBatch * D + 2 * kBatch * kRP) * sizeof(float);
    e = cudaFuncSetAttribute(attn_bwd_rows_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem_rows);
    if (e != cudaSuccess) return e;
    attn_bwd_rows_kernel<T, D><<<dim3(plan.chunks, B), kThreads, smem_rows, st>>>(
        static_cast<const T*>(C), static_cast<const T*>(dO), static_cast<T*>(dC), ws, lay, part, M, r,
        plan.rows_per_cta, flags);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (chunks > 1) {
    sum_chunks_kernel<<<dim3((2 * D * kRP + 255) / 256, B), 256, 0, st>>>(part, chunks, 2 * D * kRP);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const size_t smem_user = (size_t)(2 * D * (kRP + 1) + 2 * kRP * D + D * (D + 1)) * sizeof(float);
  e = cudaFuncSetAttribute(attn_bwd_user_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_user);
  if (e != cudaSuccess) return e;
  attn_bwd_user_kernel<T, D><<<B, kUserThreads, smem_user, st>>>(part, chunks, S, V, static_cast<const T*>(Wq),
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
