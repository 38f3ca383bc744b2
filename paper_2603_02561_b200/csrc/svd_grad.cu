// Backward pass of the truncated SVD with U absent from the forward pass (Eq. 13-15 and
// the appendix that derives them):
//   dL/dH = U [ diag(dS) + 2 Sigma sym(F o (Vbar^T V)) ] V^T,   U = H V Sigma^-1,
//   F_ij = 1 / (sigma_i^2 - sigma_j^2)  (Eq. 14), zero on the diagonal.
// The Hadamard factor is Vbar^T V: the appendix expands Tr((V^T Vbar)^T Omega_V) with the
// indices of V^T Vbar transposed, which flips the sign of the off-diagonal term; this is
// the form that agrees with finite differences of the forward pass.
//
// Because U = H V Sigma^-1, the gradient is one right-multiplication of the history,
//   dH_b = H_b K_b,   K_b = V W V^T  (d x d),   W = Sigma^-1 [ diag(dS) + Sigma (X + X^T) ],
//   X = F o (Vbar^T V),
// so the backward pass streams H once more (the same kernel that forms U Sigma = H V)
// instead of materialising U.  This file holds the per-user kernel that forms K_b.
//
// Stabilisation (the paper gives none): F_ij = D / (D^2 + eps^2) with
// D = sigma_i^2 - sigma_j^2 and eps = eps_rel * max sigma^2; eps_rel = 0 is Eq. 14 itself,
// with F_ij = 0 where D = 0.  A direction with sigma_i = 0 has no U column and gets no
// gradient (row i of W is zero).
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kGradThreads = 1024;   // latency-bound small products: many warps per scheduler

template <int D>
__global__ void __launch_bounds__(kGradThreads)
svd_grad_kernel(const float* __restrict__ S, const float* __restrict__ V, const float* __restrict__ dS,
                const float* __restrict__ dV, float eps_rel, int r, float* __restrict__ K) {
  extern __shared__ __align__(16) float sm[];
  const int lw = r | 1;                 // odd pitch: every matrix here is read along rows and along columns
  float* Vs = sm;                       // [D][lw]
  float* dVs = Vs + D * lw;             // [D][lw]  Vbar
  float* Pt = dVs + D * lw;             // [r][lw]  Vbar^T V
  float* W = Pt + r * lw;               // [r][lw]
  float* T1 = W + r * lw;               // [D][lw]  V W
  float* ss = T1 + D * lw;              // [r] sigma
  float* ds = ss + r;                   // [r] dL/dsigma
  const int b = blockIdx.x, tid = threadIdx.x;

  for (int e = tid; e < D * r; e += kGradThreads) {
    const int k = e / r, i = e % r;
    Vs[k * lw + i] = V[(size_t)b * D * r + e];
    dVs[k * lw + i] = dV[(size_t)b * D * r + e];
  }
  for (int e = tid; e < r; e += kGradThreads) { ss[e] = S[(size_t)b * r + e]; ds[e] = dS[(size_t)b * r + e]; }
  __syncthreads();

  // Pt[i][j] = sum_k Vbar[k][i] V[k][j]
  for (int e = tid; e < r * r; e += kGradThreads) {
    const int i = e / r, j = e % r;
    float acc = 0.f;
#pragma unroll 4
    for (int k = 0; k < D; ++k) acc = fmaf(dVs[k * lw + i], Vs[k * lw + j], acc);
    Pt[i * lw + j] = acc;
  }
  float smax = 0.f;
  for (int i = 0; i < r; ++i) smax = fmaxf(smax, ss[i]);
  const float eps = eps_rel * smax * smax;
  __syncthreads();

  // W = Sigma^-1 diag(dS) + (X + X^T) on the rows with sigma_i > 0
  for (int e = tid; e < r * r; e += kGradThreads) {
    const int i = e / r, j = e % r;
    const float si = ss[i], sj = ss[j];
    float w = 0.f;
    if (si > 0.f) {
      if (i == j) {
        w = ds[i] / si;
      } else {
        const float dd = (si - sj) * (si + sj);               // sigma_i^2 - sigma_j^2 without cancellation
        const float den = fmaf(dd, dd, eps * eps);
        const float f = den > 0.f ? dd / den : 0.f;
        w = f * (Pt[i * lw + j] - Pt[j * lw + i]);            // F_ij P_ij + F_ji P_ji, F skew-symmetric
      }
    }
    W[i * lw + j] = w;
  }
  __syncthreads();

  // T1 = V W  [D][r]
  for (int e = tid; e < D * r; e += kGradThreads) {
    const int k = e / r, j = e % r;
    float acc = 0.f;
#pragma unroll 4
    for (int i = 0; i < r; ++i) acc = fmaf(Vs[k * lw + i], W[i * lw + j], acc);
    T1[k * lw + j] = acc;
  }
  __syncthreads();

  // K = T1 V^T  [D][D]
  float* Kb = K + (size_t)b * D * D;
  for (int e = tid; e < D * D; e += kGradThreads) {
    const int k = e / D, l = e % D;
    float acc = 0.f;
#pragma unroll 4
    for (int j = 0; j < r; ++j) acc = fmaf(T1[k * lw + j], Vs[l * lw + j], acc);
    Kb[e] = acc;
  }
}

template <int D>
cudaError_t launch_d(int B, int r, const float* S, const float* V, const float* dS, const float* dV,
                     float eps_rel, float* K, cudaStream_t st) {
  const size_t smem = (size_t)(3 * D * (r | 1) + 2 * r * (r | 1) + 2 * r) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(svd_grad_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  svd_grad_kernel<D><<<B, kGradThreads, smem, st>>>(S, V, dS, dV, eps_rel, r, K);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_svd_grad(int B, int d, int r, const float* S, const float* V, const float* dS,
                            const float* dV, float eps_rel, float* K, cudaStream_t st) {
  switch (d) {
    case 32: return launch_d<32>(B, r, S, V, dS, dV, eps_rel, K, st);
    case 64: return launch_d<64>(B, r, S, V, dS, dV, eps_rel, K, st);
    case 128: return launch_d<128>(B, r, S, V, dS, dV, eps_rel, K, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace solar
