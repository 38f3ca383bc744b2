// Batched symmetric eigensolver: G_b = V Lambda V^T by parallel two-sided Jacobi
// rotations in shared memory, one CTA per user.  The top-r eigenpairs give the
// truncated SVD of Eq. 9 without U: s_i = sqrt(lambda_i), v_i = eigenvector.
//
// Parallel ordering: round-robin tournament (D/2 disjoint pairs per round, D-1
// rounds per sweep).  In one round every 2x2 block G[{p,q}][{p',q'}] is touched
// by exactly one thread, which applies the row pair's rotation from the left and
// the column pair's from the right.  Each thread recomputes the (at most four)
// rotations it needs from the diagonal blocks of the current matrix, and the
// matrix is double-buffered, so a round costs ONE block barrier.
#include <math.h>

#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr float kTolRel = 2.3841858e-07f;  // 2^-22: |g_pq| <= tol*sqrt(g_pp g_qq) counts as zero
constexpr float kTolAbs = 7.4505806e-09f;  // 2^-27 of the largest diagonal entry

template <int D> struct EigCfg {
  static constexpr int NP = D / 2;                 // pairs per round
  static constexpr int PT = (D == 128) ? 2 : 1;    // row pairs (and column pairs) per thread
  static constexpr int SIDE = NP / PT;             // threads along each side of the block grid
  static constexpr int THREADS = SIDE * SIDE;
  static constexpr int LD = D + 1;
  static constexpr size_t SMEM = (size_t)(3 * D * LD + 2 * D) * sizeof(float);
};

// Pair i of round k in the circle method on n players (n even): every unordered
// pair meets exactly once in rounds 0..n-2.
__device__ __forceinline__ void pair_of(int k, int i, int n, int& p, int& q) {
  int a, c;
  if (i == 0) {
    a = n - 1; c = k;
  } else {
    a = k + i;       if (a >= n - 1) a -= n - 1;
    c = k - i;       if (c < 0) c += n - 1;
  }
  p = min(a, c); q = max(a, c);
}

// Rotation J = [[c, s], [-s, c]] that annihilates g_pq of the 2x2 symmetric block
// [[a, g], [g, b]]; identity when g is negligible (or not a number).  Returned
// as s, tau = s/(1+c) and t = s/c: columns are updated in the cancellation-free
// form x_p' = x_p - s (x_q + tau x_p), x_q' = x_q + s (x_p - tau x_q), and the
// diagonal as a' = a - t g, b' = b + t g, so a near-identity rotation perturbs
// the matrix by O(s) instead of by a rounding error of the full entry.
struct Rot { float s, tau, t; };

__device__ __forceinline__ Rot jacobi_rot(float a, float b, float g, float thr_abs) {
  const float ag = fabsf(g);
  const bool act = (ag > thr_abs) && (ag > kTolRel * sqrtf(fabsf(a * b)));
  const float dlt = b - a;
  const float h = sqrtf(fmaf(dlt, dlt, 4.f * g * g));
  // t = tan(theta) = sgn(zeta) / (|zeta| + sqrt(1 + zeta^2)),  zeta = (b - a) / (2 g)
  const float t = __fdividef(copysignf(2.f * g, dlt * g), fabsf(dlt) + h);
  const float c = rsqrtf(fmaf(t, t, 1.f));
  const float s = t * c;
  Rot r;
  r.s = act ? s : 0.f;
  r.t = act ? t : 0.f;
  r.tau = act ? __fdividef(s, 1.f + c) : 0.f;
  return r;
}

__device__ __forceinline__ void rot_apply(const Rot& r, float& xp, float& xq) {
  const float p = xp, q = xq;
  xp = fmaf(-r.s, fmaf(r.tau, p, q), p);
  xq = fmaf(r.s, fmaf(-r.tau, q, p), q);
}

template <int D>
__global__ void __launch_bounds__(EigCfg<D>::THREADS, 1)
eig_jacobi_kernel(const float* __restrict__ gpart, int splits, int r, float* __restrict__ S,
                  float* __restrict__ V, int* __restrict__ info) {
  using Cfg = EigCfg<D>;
  constexpr int PT = Cfg::PT, SIDE = Cfg::SIDE, LD = Cfg::LD, NT = Cfg::THREADS;
  extern __shared__ float smem[];
  float* Gc = smem;                 // current matrix
  float* Gn = smem + D * LD;        // next matrix
  float* Vm = smem + 2 * D * LD;    // accumulated rotations (eigenvectors in columns)
  float* lam = smem + 3 * D * LD;   // [D] eigenvalues
  int* order = reinterpret_cast<int*>(lam + D);   // [D] column holding the k-th largest eigenvalue
  __shared__ float s_gmax;

  const int b = blockIdx.x, tid = threadIdx.x;
  const int tI = tid / SIDE, tJ = tid % SIDE;

  // ---- G = sum of the slices' partial Grams, in slice order -----------------
  const float* gp = gpart + (size_t)b * splits * D * D;
  int bad = 0;
  for (int e = tid; e < D * D; e += NT) {
    double acc = 0.0;
    for (int s = 0; s < splits; ++s) acc += (double)gp[(size_t)s * D * D + e];
    const float g = (float)acc;
    bad |= !isfinite(g);
    const int i = e / D, j = e % D;
    Gc[i * LD + j] = g;
    Vm[i * LD + j] = (i == j) ? 1.f : 0.f;
  }
  bad = __syncthreads_or(bad);
  if (bad) {
    const float qnan = __int_as_float(0x7fc00000);
    for (int e = tid; e < D * r; e += NT) V[(size_t)b * D * r + e] = qnan;
    for (int e = tid; e < r; e += NT) S[(size_t)b * r + e] = qnan;
    if (tid == 0 && info) info[b] = SOLAR_INFO_NONFINITE;
    return;
  }
  if (tid < 32) {
    float m = 0.f;
    for (int i = tid; i < D; i += 32) m = fmaxf(m, fabsf(Gc[i * LD + i]));
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (tid == 0) s_gmax = m;
  }
  __syncthreads();
  const float thr_abs = kTolAbs * s_gmax;

  // ---- sweeps -----------------------------------------------------------------
  int converged = 0;
  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    int rotated = 0;
    for (int k = 0; k < D - 1; ++k) {
      int pr[PT], qr[PT], pc[PT], qc[PT];
      Rot rr[PT], rc[PT];
#pragma unroll
      for (int a = 0; a < PT; ++a) {
        pair_of(k, tI + a * SIDE, D, pr[a], qr[a]);
        rr[a] = jacobi_rot(Gc[pr[a] * LD + pr[a]], Gc[qr[a] * LD + qr[a]], Gc[pr[a] * LD + qr[a]],
                           thr_abs);
        pair_of(k, tJ + a * SIDE, D, pc[a], qc[a]);
        rc[a] = jacobi_rot(Gc[pc[a] * LD + pc[a]], Gc[qc[a] * LD + qc[a]], Gc[pc[a] * LD + qc[a]],
                           thr_abs);
        rotated |= (rc[a].s != 0.f);
      }
#pragma unroll
      for (int a = 0; a < PT; ++a) {
#pragma unroll
        for (int c = 0; c < PT; ++c) {
          // G' = J_row^T G J_col on the block rows (p,q) x columns (p',q')
          float x00 = Gc[pr[a] * LD + pc[c]], x01 = Gc[pr[a] * LD + qc[c]];
          float x10 = Gc[qr[a] * LD + pc[c]], x11 = Gc[qr[a] * LD + qc[c]];
          if (pr[a] == pc[c]) {            // the pair's own diagonal block
            const float tg = rc[c].t * x01;
            x00 -= tg; x11 += tg;
            if (rc[c].s != 0.f) { x01 = 0.f; x10 = 0.f; }
          } else {
            rot_apply(rc[c], x00, x01); rot_apply(rc[c], x10, x11);   // columns
            rot_apply(rr[a], x00, x10); rot_apply(rr[a], x01, x11);   // rows
          }
          Gn[pr[a] * LD + pc[c]] = x00; Gn[pr[a] * LD + qc[c]] = x01;
          Gn[qr[a] * LD + pc[c]] = x10; Gn[qr[a] * LD + qc[c]] = x11;
          // V' = V J_col on fixed rows (2I, 2I+1)
          const int r0 = 2 * (tI + a * SIDE);
          float v00 = Vm[r0 * LD + pc[c]], v01 = Vm[r0 * LD + qc[c]];
          float v10 = Vm[(r0 + 1) * LD + pc[c]], v11 = Vm[(r0 + 1) * LD + qc[c]];
          rot_apply(rc[c], v00, v01); rot_apply(rc[c], v10, v11);
          Vm[r0 * LD + pc[c]] = v00; Vm[r0 * LD + qc[c]] = v01;
          Vm[(r0 + 1) * LD + pc[c]] = v10; Vm[(r0 + 1) * LD + qc[c]] = v11;
        }
      }
      __syncthreads();
      float* t = Gc; Gc = Gn; Gn = t;
    }
    if (!__syncthreads_or(rotated)) { converged = 1; break; }
  }

  // ---- order the eigenvalues, keep r, fix the sign of each vector ----------------
  if (tid < D) lam[tid] = Gc[tid * LD + tid];
  __syncthreads();
  if (tid < D) {
    const float li = lam[tid];
    int rank = 0;
    for (int j = 0; j < D; ++j) {
      const float lj = lam[j];
      rank += (lj > li) || (lj == li && j < tid);
    }
    order[rank] = tid;
  }
  __syncthreads();
  float* sgn = Gn;   // reuse: [r] signs
  if (tid < r) {
    const int col = order[tid];
    float best = -1.f, lead = 1.f;
    for (int j = 0; j < D; ++j) {
      const float v = Vm[j * LD + col];
      if (fabsf(v) > best) { best = fabsf(v); lead = v; }   // strict: lowest index wins a tie
    }
    sgn[tid] = lead < 0.f ? -1.f : 1.f;
    S[(size_t)b * r + tid] = sqrtf(fmaxf(lam[col], 0.f));
  }
  __syncthreads();
  for (int e = tid; e < D * r; e += NT) {
    const int j = e / r, i = e % r;
    V[(size_t)b * D * r + e] = Vm[j * LD + order[i]] * sgn[i];
  }
  if (tid == 0 && info) info[b] = converged ? 0 : SOLAR_INFO_NOT_CONVERGED;
}

template <int D>
cudaError_t launch_d(int B, int r, const float* gpart, int splits, float* S, float* V, int* info,
                     cudaStream_t st) {
  using Cfg = EigCfg<D>;
  cudaError_t e = cudaFuncSetAttribute(eig_jacobi_kernel<D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::SMEM);
  if (e != cudaSuccess) return e;
  eig_jacobi_kernel<D><<<B, Cfg::THREADS, Cfg::SMEM, st>>>(gpart, splits, r, S, V, info);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_eig_jacobi(int B, int d, int r, const float* gpart, int splits, float* S,
                              float* V, int* info, cudaStream_t st) {
  switch (d) {
    case 32: return launch_d<32>(B, r, gpart, splits, S, V, info, st);
    case 64: return launch_d<64>(B, r, gpart, splits, S, V, info, st);
    case 128: return launch_d<128>(B, r, gpart, splits, S, V, info, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace solar
