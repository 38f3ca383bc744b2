// Batched symmetric eigensolver for the Gram matrices: G_b = V Lambda V^T, top-r
// pairs only, one CTA per user, everything in shared memory.  The top-r
// eigenpairs give the truncated SVD of Eq. 9 without U: s_i = sqrt(lambda_i).
//
// Two routes inside the one kernel:
//
//  (1) Subspace route -- Algorithm 1 (randomized range finder with power
//      iteration) applied to the Gram matrix: Omega is Gaussian, each power step
//      is Y = G Z followed by a Cholesky-QR in double precision, and the small
//      SVD at the end of Algorithm 1 becomes the p x p Rayleigh-Ritz problem
//      T = Z^T G Z, solved by parallel two-sided Jacobi (p = 8, 16 or 32 >= r).
//      The result is accepted only if it is CERTIFIED a posteriori: the residuals
//      G v_i - theta_i v_i must be small against the gaps of the Ritz values, and
//      the trace of G must show that nothing outside the kept r pairs can reach
//      theta_r.  Otherwise the CTA falls through to route (2).
//
//  (2) Full route -- parallel two-sided Jacobi on the whole d x d matrix, always
//      valid (Eq. 9's exact truncated SVD for any spectrum).
//
// Both Jacobi solves use the round-robin tournament in systolic form: the matrix is
// indexed by slot, the pairs of every round are the slots (2i, 2i+1), and a fixed slot
// move after each round makes every two indices meet once in n-1 rounds.  In one round
// every 2x2 block is touched by exactly one thread, which applies the row pair's rotation
// from the left and the column pair's from the right; each thread recomputes the
// rotations it needs from the diagonal blocks of the current matrix, and the matrix is
// double-buffered, so a round costs ONE barrier.  The 2x2 blocks are stored in four
// planes so that every access of a warp is free of bank conflicts.
#include "eig_jacobi.cuh"

namespace solar {

namespace {

constexpr int kMaxSubspaceIters = 5;       // power steps before the subspace route gives up

// Acceptance thresholds of the subspace route (chosen by the storage type).
struct EigTol {
  float eps_vec;     // certified bound on sin(angle) of every kept vector
  float floor_rel;   // residuals below floor_rel*theta_1 are at the rounding level of fp32
  float sweep_stop;  // a Jacobi sweep whose largest relative off-diagonal was below this is the last
};

template <int D> struct EigCfg {
  // d = 32 and d = 64 run on 256 threads (1 and 4 blocks per thread in the full route), so
  // that a CTA leaves registers and shared memory for other kernels' CTAs on its SM;
  // d = 128 needs 1024 (4 blocks per thread)
  static constexpr int THREADS = (D == 128) ? 1024 : 256;
  static constexpr int LD = D + 4;                 // rows stay 16-byte aligned
  static constexpr int PMAX = (D >= 64) ? 32 : 16; // largest subspace dimension (<= D/2)
  static constexpr int LP = PMAX + 1;
  static constexpr int LPD = PMAX + 2;             // row pitch of the double matrices (16-byte rows)
  // floats of the full route: Gc, Gn, Vm, lam[D], order[D], perm[2][D]
  static constexpr int FULL_FLOATS = 3 * D * LD + 4 * D;
  // floats of the subspace route: Ad, Li [PMAX][LPD], dref [PMAX] (double, first: 16-byte aligned),
  // Zb, Yb, Xb [D][PMAX], Tc, Wm [PMAX][LP], theta, res2, ordp [PMAX], pad; Tb, Wb [2][PMAX*(PMAX+2)] lie over Ad, Li
  static constexpr int SUB_FLOATS = 2 * (2 * PMAX * LPD + PMAX) + 3 * D * PMAX + 2 * PMAX * LP +
                                    3 * PMAX + 3;
  static_assert(4 * PMAX * (PMAX + 2) <= 2 * (2 * PMAX * LPD + PMAX), "Tb, Wb must fit over Ad, Li, dref");
  // The [D][PMAX] buffers of the subspace route always alias Gn and Vm (free until the full
  // route starts); for D = 128 so do all the others.
  static constexpr bool ALIAS = (D == 128);
  static constexpr int DPM_FLOATS = 3 * D * PMAX;
  static constexpr size_t SMEM =
      (size_t)(FULL_FLOATS + (ALIAS ? 0 : SUB_FLOATS - DPM_FLOATS)) * sizeof(float);
  static_assert(!ALIAS || SUB_FLOATS <= 2 * D * LD, "subspace buffers must fit in Gn+Vm");
  static_assert(DPM_FLOATS <= 2 * D * LD && DPM_FLOATS % 4 == 0, "Zb, Yb, Xb must fit in Gn+Vm");
  static_assert((D * LD) % 4 == 0 && FULL_FLOATS % 4 == 0, "16-byte alignment of the regions");
};

// Integer mixer (two multiply-xorshift rounds) used as a counter-based generator.
__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7feb352du;
  x ^= x >> 15; x *= 0x846ca68bu;
  x ^= x >> 16;
  return x;
}

// Entry e of the Gaussian test matrix Omega of Algorithm 1 (Box-Muller on two
// counter-derived uniforms); the same matrix for every user and every call.
__device__ __forceinline__ float omega_entry(uint32_t e) {
  const float u1 = ((float)(mix32(2u * e + 0x9e3779b9u) >> 8) + 0.5f) * (1.f / 16777216.f);
  const float u2 = ((float)(mix32(2u * e + 0x85ebca6bu) >> 8) + 0.5f) * (1.f / 16777216.f);
  return sqrtf(-2.f * __logf(u1)) * __cosf(6.2831853f * u2);
}

// 1/sqrt(x) in double: the fp32 approximation (relative error 2^-22) and ONE Newton step
// in double (2^-43).  That is ample for the Cholesky-QR -- a relative error e in a pivot's
// inverse root scales one column of Q by 1 + e -- and every double-precision operation here
// sits on the 32-step critical path of the factorisation.
__device__ __forceinline__ double rsqrt_f64(double x) {
  const double y = (double)rsqrtf((float)x);
  return fma(y, fma(-0.5 * x * y, y, 0.5), y);
}

// ---- small dense products in shared memory -------------------------------------------

// Out[D][p] = G Z.  G is [D][LD] (symmetric), Z and Out are [D][p], p even.
// Each thread owns a 4 x 2 tile: four 16-byte reads of G rows and four 8-byte
// reads of Z feed 32 FMAs, so the loop is not bound by shared-memory issue.
template <int D, int LD>
__device__ __forceinline__ void mul_G(const float* __restrict__ G, const float* __restrict__ Z,
                                      float* __restrict__ Out, int p, int tid, int nt) {
  const int cp = p >> 1;
  const int ntiles = (D / 4) * cp;
  for (int t = tid; t < ntiles; t += nt) {
    const int j0 = (t % cp) * 2, i0 = (t / cp) * 4;
    float acc[4][2];
#pragma unroll
    for (int m = 0; m < 4; ++m) { acc[m][0] = 0.f; acc[m][1] = 0.f; }
#pragma unroll 2
    for (int k = 0; k < D; k += 4) {
      float4 g[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) g[m] = *reinterpret_cast<const float4*>(G + (i0 + m) * LD + k);
      const float2 z0 = *reinterpret_cast<const float2*>(Z + (k + 0) * p + j0);
      const float2 z1 = *reinterpret_cast<const float2*>(Z + (k + 1) * p + j0);
      const float2 z2 = *reinterpret_cast<const float2*>(Z + (k + 2) * p + j0);
      const float2 z3 = *reinterpret_cast<const float2*>(Z + (k + 3) * p + j0);
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        acc[m][0] = fmaf(g[m].x, z0.x, acc[m][0]); acc[m][1] = fmaf(g[m].x, z0.y, acc[m][1]);
        acc[m][0] = fmaf(g[m].y, z1.x, acc[m][0]); acc[m][1] = fmaf(g[m].y, z1.y, acc[m][1]);
        acc[m][0] = fmaf(g[m].z, z2.x, acc[m][0]); acc[m][1] = fmaf(g[m].z, z2.y, acc[m][1]);
        acc[m][0] = fmaf(g[m].w, z3.x, acc[m][0]); acc[m][1] = fmaf(g[m].w, z3.y, acc[m][1]);
      }
    }
#pragma unroll
    for (int m = 0; m < 4; ++m)
      *reinterpret_cast<float2*>(Out + (i0 + m) * p + j0) = make_float2(acc[m][0], acc[m][1]);
  }
}

// Out[a][c] = sum_k X[k][a] Y[k][c] over the D rows; X, Y are [D][p]; Out is [p][ldo].
// 2 x 2 tile per thread, accumulation in Acc (double for the Cholesky-QR Gram matrix).
template <int D, typename Acc, typename OutT>
__device__ __forceinline__ void mul_XtY(const float* __restrict__ X, const float* __restrict__ Y,
                                        OutT* __restrict__ Out, int p, int ldo, int tid, int nt) {
  const int cp = p >> 1;
  for (int t = tid; t < cp * cp; t += nt) {
    const int c0 = (t % cp) * 2, a0 = (t / cp) * 2;
    Acc s00 = 0, s01 = 0, s10 = 0, s11 = 0;
#pragma unroll 4
    for (int k = 0; k < D; ++k) {
      const float2 x = *reinterpret_cast<const float2*>(X + k * p + a0);
      const float2 y = *reinterpret_cast<const float2*>(Y + k * p + c0);
      s00 += (Acc)x.x * (Acc)y.x; s01 += (Acc)x.x * (Acc)y.y;
      s10 += (Acc)x.y * (Acc)y.x; s11 += (Acc)x.y * (Acc)y.y;
    }
    Out[a0 * ldo + c0] = (OutT)s00;       Out[a0 * ldo + c0 + 1] = (OutT)s01;
    Out[(a0 + 1) * ldo + c0] = (OutT)s10; Out[(a0 + 1) * ldo + c0 + 1] = (OutT)s11;
  }
}

// Cholesky A = L L^T of the p x p matrix A (double, [p][ld], ld even; the lower triangle
// is overwritten by L) fused with the inverse Li = L^{-1} ([p][ld], upper part zero), by
// ONE warp.  Lane j owns row j of L and column j of Li.  Step k computes column k of L
// (a dot of row j with row k) and row k of Li (a dot of row k of L with column j of Li):
// both use the same broadcast row of L, so the inverse rides in the latency shadow of the
// factorisation.  A numerically dependent column (pivot below 1e-13 of its original diagonal
// entry) is deflated: its column of L and row of Li are zero, so Q gets a zero column there.
// Returns false (uniformly) only for a non-finite pivot.
__device__ __forceinline__ bool cholesky_inverse_warp(double* __restrict__ A,
                                                      double* __restrict__ Li,
                                                      double* __restrict__ dref, int p, int ld,
                                                      int lane) {
  const int j = lane < p ? lane : 0;        // surplus lanes shadow lane 0 and store nothing
  const bool mine = lane < p;
  const double* row = A + j * ld;
  if (mine) dref[j] = row[j];                // original diagonal: the yardstick of the pivots
  __syncwarp();
  for (int k = 0; k < p; ++k) {
    const double* rk = A + k * ld;
    double c0 = row[k], c1 = 0.0;
    double e0 = (j == k) ? 1.0 : 0.0, e1 = 0.0;
    int i = 0;
    double c2 = 0.0, c3 = 0.0, e2 = 0.0, e3 = 0.0;
#pragma unroll 2
    for (; i + 3 < k; i += 4) {              // all ten loads of a 4-wide step are independent
      const double2 lk0 = *reinterpret_cast<const double2*>(rk + i);
      const double2 lk1 = *reinterpret_cast<const double2*>(rk + i + 2);
      const double2 lj0 = *reinterpret_cast<const double2*>(row + i);
      const double2 lj1 = *reinterpret_cast<const double2*>(row + i + 2);
      const double x0 = Li[i * ld + j], x1 = Li[(i + 1) * ld + j];
      const double x2 = Li[(i + 2) * ld + j], x3 = Li[(i + 3) * ld + j];
      c0 = fma(-lj0.x, lk0.x, c0); c1 = fma(-lj0.y, lk0.y, c1);
      c2 = fma(-lj1.x, lk1.x, c2); c3 = fma(-lj1.y, lk1.y, c3);
      e0 = fma(-lk0.x, x0, e0);    e1 = fma(-lk0.y, x1, e1);
      e2 = fma(-lk1.x, x2, e2);    e3 = fma(-lk1.y, x3, e3);
    }
    c0 += c2; c1 += c3; e0 += e2; e1 += e3;
    for (; i + 1 < k; i += 2) {
      const double2 lk = *reinterpret_cast<const double2*>(rk + i);
      const double2 lj = *reinterpret_cast<const double2*>(row + i);
      const double x0 = Li[i * ld + j], x1 = Li[(i + 1) * ld + j];
      c0 = fma(-lj.x, lk.x, c0); c1 = fma(-lj.y, lk.y, c1);
      e0 = fma(-lk.x, x0, e0);   e1 = fma(-lk.y, x1, e1);
    }
    if (i < k) {
      const double lk = rk[i];
      c0 = fma(-row[i], lk, c0);
      e0 = fma(-lk, Li[i * ld + j], e0);
    }
    const double c = c0 + c1;
    const double piv = __shfl_sync(0xffffffffu, c, k);
    const double ref = dref[k];
    if (!(piv < 1e300)) return false;                    // NaN or overflow
    // A column whose part orthogonal to the earlier ones is below 3e-7 of its length is
    // rounding residue (Y is fp32) of a rank-deficient block: it is dropped (zero column
    // of Q).  Above that the direction may be noisy but Q stays orthonormal: the
    // arithmetic here is double, and any orthonormal basis serves the Rayleigh-Ritz step.
    const double inv = (piv > 1e-13 * ref) ? rsqrt_f64(piv) : 0.0;
    if (mine && j >= k) A[j * ld + k] = c * inv;
    if (mine) Li[k * ld + j] = (j <= k) ? (e0 + e1) * inv : 0.0;
    __syncwarp();
  }
  return true;
}

// Z[i][j] = sum_{k<=j} Y[i][k] Li[j][k]  (Z = Y L^{-T}: the Q factor of the Cholesky-QR).
// Two rows per thread share each 16-byte read of Li.
template <int D>
__device__ __forceinline__ void apply_Linv_t(const float* __restrict__ Y,
                                             const double* __restrict__ Li, float* __restrict__ Z,
                                             int p, int ld, int tid, int nt) {
  for (int t = tid; t < (D / 2) * p; t += nt) {
    const int j = t % p, i0 = (t / p) * 2;
    double s0 = 0.0, s1 = 0.0, u0 = 0.0, u1 = 0.0;
#pragma unroll 4
    for (int k = 0; k < p; k += 2) {      // Li[j][k] = 0 for k > j
      const double2 l = *reinterpret_cast<const double2*>(Li + j * ld + k);
      const float2 ya = *reinterpret_cast<const float2*>(Y + i0 * p + k);
      const float2 yb = *reinterpret_cast<const float2*>(Y + (i0 + 1) * p + k);
      s0 = fma((double)ya.x, l.x, s0); s1 = fma((double)ya.y, l.y, s1);
      u0 = fma((double)yb.x, l.x, u0); u1 = fma((double)yb.y, l.y, u1);
    }
    Z[i0 * p + j] = (float)(s0 + s1);
    Z[(i0 + 1) * p + j] = (float)(u0 + u1);
  }
}

// acc[m] = sum_k X[i0+m][k] M[k][col], m = 0..R-1: R rows of X ([.][p], 16-byte reads)
// against one column of M ([p][ldm]).
template <int R>
__device__ __forceinline__ void rows_dot_col(const float* __restrict__ X, const float* __restrict__ M,
                                             int p, int ldm, int i0, int col, float (&acc)[R]) {
#pragma unroll
  for (int m = 0; m < R; ++m) acc[m] = 0.f;
#pragma unroll 2
  for (int k = 0; k < p; k += 4) {
    const float m0 = M[(k + 0) * ldm + col], m1 = M[(k + 1) * ldm + col];
    const float m2 = M[(k + 2) * ldm + col], m3 = M[(k + 3) * ldm + col];
#pragma unroll
    for (int m = 0; m < R; ++m) {
      const float4 x = *reinterpret_cast<const float4*>(X + (i0 + m) * p + k);
      acc[m] = fmaf(x.x, m0, acc[m]); acc[m] = fmaf(x.y, m1, acc[m]);
      acc[m] = fmaf(x.z, m2, acc[m]); acc[m] = fmaf(x.w, m3, acc[m]);
    }
  }
}

// ---- Jacobi on the p x p Rayleigh-Ritz matrix ------------------------------------------
// Same systolic tournament as the full route (slot_next), on the small matrix.
// Layout of the Ritz Jacobi (thread (I, J) = tid / hp, tid % hp: a warp holds 32 / hp whole
// rows of blocks): row pitch hp and a plane stride of hp * hp plus a small offset.  An
// exhaustive count over all 18 shared-memory accesses of a round (own block, the two diagonal
// blocks, the eight scattered writes) gives for p = 32: every access free of bank conflicts but
// six per round and CTA, where the pitch hp + 1 of blk_off leaves twelve of the eighteen two-way
// conflicted (consecutive rows overlap in one bank); the offsets for the smaller p come from
// the same count.
__device__ __forceinline__ int rplane(int hp) { return hp * hp + (hp == 12 ? 18 : hp == 4 ? 6 : 2); }
__device__ __forceinline__ int rblk_off(int u, int v, int hp) {
  return (((u & 1) << 1) + (v & 1)) * rplane(hp) + (u >> 1) * hp + (v >> 1);
}
__device__ __forceinline__ int rblk_size(int hp) { return 4 * rplane(hp); }

// Run by the first jt = roundup((p/2)^2, 32) threads of the CTA (barrier id 1).  Thread
// (I, J) of the (p/2) x (p/2) grid owns block (I, J) of T and of W in every round: it reads
// its block, the two diagonal blocks that define its row and column rotation, and its W
// block, and writes the eight rotated entries to destinations fixed once per thread (the
// slot move).  T and W are double-buffered ([2][blk_size] each; buffer 0 holds the input, W
// the identity).  Returns the sweeps used (negative: cap reached); the result is in buffer
// (sweeps*(p-1)) & 1.
__device__ __forceinline__ int ritz_jacobi(float* Tb, float* Wb, int p, float thr_abs2,
                                           float sweep_stop2, volatile int* flags, int tid, int jt) {
  const int hp = p >> 1;
  const int plane = rplane(hp), bufsz = 4 * plane;
  const bool active = tid < hp * hp;
  const int I = active ? tid / hp : 0, J = active ? tid % hp : 0;
  const int src = I * hp + J, srcI = I * hp + I, srcJ = J * hp + J;
  const int r0 = slot_next(2 * I, p), r1 = slot_next(2 * I + 1, p);
  const int c0 = slot_next(2 * J, p), c1 = slot_next(2 * J + 1, p);
  const int t00 = rblk_off(r0, c0, hp), t01 = rblk_off(r0, c1, hp);
  const int t10 = rblk_off(r1, c0, hp), t11 = rblk_off(r1, c1, hp);
  const int w00 = rblk_off(2 * I, c0, hp), w01 = rblk_off(2 * I, c1, hp);   // W's rows stay put
  const int w10 = rblk_off(2 * I + 1, c0, hp), w11 = rblk_off(2 * I + 1, c1, hp);
  int sweeps = -kMaxSweeps;
  int cur = 0;
  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    if (tid == 0) flags[(sweep + 1) % 3] = 0;
    bool worst = false;
    for (int k = 0; k < p - 1; ++k) {
      if (active) {
        const float* Tc = Tb + cur * bufsz;
        const float* Wc = Wb + cur * bufsz;
        float* Tn = Tb + (cur ^ 1) * bufsz;
        float* Wn = Wb + (cur ^ 1) * bufsz;
        bool big_r, big_c;
        const Rot rr = jacobi_rot(Tc[srcI], Tc[3 * plane + srcI], Tc[plane + srcI], thr_abs2, sweep_stop2, big_r);
        const Rot rc = jacobi_rot(Tc[srcJ], Tc[3 * plane + srcJ], Tc[plane + srcJ], thr_abs2, sweep_stop2, big_c);
        worst |= big_c;
        float x00 = Tc[src], x01 = Tc[plane + src], x10 = Tc[2 * plane + src], x11 = Tc[3 * plane + src];
        float v00 = Wc[src], v01 = Wc[plane + src], v10 = Wc[2 * plane + src], v11 = Wc[3 * plane + src];
        if (I == J) {                      // the pair's own diagonal block
          const float tg = rc.t * x01;
          x00 -= tg; x11 += tg;
          if (rc.s != 0.f) { x01 = 0.f; x10 = 0.f; }
        } else {
          rot_apply(rc, x00, x01); rot_apply(rc, x10, x11);   // columns
          rot_apply(rr, x00, x10); rot_apply(rr, x01, x11);   // rows
        }
        rot_apply(rc, v00, v01); rot_apply(rc, v10, v11);
        Tn[t00] = x00; Tn[t01] = x01; Tn[t10] = x10; Tn[t11] = x11;
        Wn[w00] = v00; Wn[w01] = v01; Wn[w10] = v10; Wn[w11] = v11;
      }
      if (k == p - 2 && worst) flags[sweep % 3] = 1;
      bar_named(1, jt);
      cur ^= 1;
    }
    if (flags[sweep % 3] == 0) { sweeps = sweep + 1; break; }
  }
  return sweeps;
}

template <int D>
__global__ void __launch_bounds__(EigCfg<D>::THREADS, 1)
eig_kernel(const float* __restrict__ gpart, const int* __restrict__ gram_status, int parts, int splits, int r,
           int p, int route, int sweep_cap, int force_iters, EigTol tol, float* __restrict__ S,
           float* __restrict__ V, int* __restrict__ info, int* __restrict__ route_taken) {
  using Cfg = EigCfg<D>;
  constexpr int LD = Cfg::LD, NT = Cfg::THREADS;
  extern __shared__ __align__(16) float smem[];
  float* Gc = smem;                 // current matrix
  float* Gn = smem + D * LD;        // next matrix
  __shared__ float s_gmax;
  __shared__ double s_trace;
  __shared__ int s_flags[4];
  __shared__ int s_sweeps;
  __shared__ int s_why;     // why the subspace route was not accepted (kWhy* bits)

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  pdl_wait();          // everything below reads what the Gram kernel wrote

  // ---- G = sum of the slices' partial Grams, in slice order -----------------
  const float4* gp = reinterpret_cast<const float4*>(gpart + (size_t)b * parts * D * D);
  // a Gram CTA whose bounded wait ran out leaves a code other than kGramStatusOk
  int lost = 0;
  for (int s = tid; s < splits; s += NT) lost |= (gram_status[b * splits + s] != kGramStatusOk);
  int bad = 0;
  for (int e = tid; e < D * D / 4; e += NT) {
    // fp32 sums in a fixed order (GW slices at a time, pairwise within the group): the
    // partials are fp32 to begin with, and one rounding per level is far below their own error.
    // All loads of a group are issued before the first add: the loop is bound by their latency.
    constexpr int GW = (D == 128) ? 8 : 16;      // 1024 threads leave 64 registers each at d = 128
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < parts; s += GW) {
      float4 v[GW];
#pragma unroll
      for (int u = 0; u < GW; ++u)
        v[u] = (s + u < parts) ? __ldg(gp + (size_t)(s + u) * (D * D / 4) + e)
                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int h = GW / 2; h >= 1; h >>= 1)
#pragma unroll
        for (int u = 0; u < h; ++u) {
          v[u].x += v[u + h].x; v[u].y += v[u + h].y; v[u].z += v[u + h].z; v[u].w += v[u + h].w;
        }
      acc.x += v[0].x; acc.y += v[0].y; acc.z += v[0].z; acc.w += v[0].w;
    }
    bad |= !(isfinite(acc.x) && isfinite(acc.y) && isfinite(acc.z) && isfinite(acc.w));
    *reinterpret_cast<float4*>(Gc + (e / (D / 4)) * LD + (e % (D / 4)) * 4) = acc;
  }
  if (tid < 4) s_flags[tid] = 0;
  if (tid == 0) { s_why = 0; s_sweeps = 0; }
  lost = __syncthreads_or(lost);
  bad = __syncthreads_or(bad);
  if (bad || lost) {
    const float qnan = __int_as_float(0x7fc00000);
    for (int e = tid; e < D * r; e += NT) V[(size_t)b * D * r + e] = qnan;
    for (int e = tid; e < r; e += NT) S[(size_t)b * r + e] = qnan;
    if (tid == 0 && info) info[b] = lost ? SOLAR_INFO_DEVICE_WAIT : SOLAR_INFO_NONFINITE;
    if (tid == 0 && route_taken) route_taken[b] = 0;
    return;
  }
  if (tid < 32) {
    float m = 0.f;
    double tr = 0.0;
    for (int i = tid; i < D; i += 32) {
      const float g = Gc[i * LD + i];
      m = fmaxf(m, fabsf(g));
      tr += (double)g;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      tr += __shfl_xor_sync(0xffffffffu, tr, o);
    }
    if (tid == 0) { s_gmax = m; s_trace = tr; }
  }
  __syncthreads();
  const float gmax = s_gmax;
  // Power-of-two scale that brings the largest diagonal entry into [1, 2): everything
  // below works on sc * G (exact), and the eigenvalues are divided by sc at the end.
  const float sc = gmax > 0.f ? exp2f(-(float)max(-100, min(100, ilogbf(gmax)))) : 1.f;
  for (int e = tid; e < D * D; e += NT) Gc[(e / D) * LD + (e % D)] *= sc;
  __syncthreads();
  const float thr_abs2 = (kTolAbs * gmax * sc) * (kTolAbs * gmax * sc);
  const float stop2 = tol.sweep_stop * tol.sweep_stop;

  // ======================= route (1): certified subspace iteration =======================
  if (p > 0 && route != kRouteFull && gmax > 0.f) {
    constexpr int LP = Cfg::LP, PM = Cfg::PMAX;
    float* sub = Cfg::ALIAS ? Gn + Cfg::DPM_FLOATS : smem + Cfg::FULL_FLOATS;
    constexpr int LPD = Cfg::LPD;
    double* Ad = reinterpret_cast<double*>(sub);          // [PM][LPD] Y^T Y, then its Cholesky factor
    double* Li = Ad + PM * LPD;                           // [PM][LPD] inverse of the factor
    double* dref = Li + PM * LPD;                         // [PM]      diagonal of Y^T Y
    float* Zb = Gn;                                       // [D][p]    orthonormal basis (over Gn, Vm)
    float* Yb = Zb + D * PM;                              // [D][p]    G Z
    float* Xb = Yb + D * PM;                              // [D][p]    scratch / Ritz vectors
    float* Tc = reinterpret_cast<float*>(dref + PM);      // [p][LP]
    float* Wm = Tc + PM * LP;                             // [p][LP]   Ritz eigenvectors, row-major
    // The Jacobi's buffers lie over Ad, Li, dref: the Cholesky-QR is over when T is packed
    // into them, and they are unpacked into Wm and theta before a retry orthonormalises again.
    float* Tb = reinterpret_cast<float*>(Ad);             // [2][blk_size] Jacobi matrix, two buffers
    float* Wb = Tb + 2 * PM * (PM + 2);                   // [2][blk_size] accumulated rotations
    float* theta = Wm + PM * LP;                          // [p]
    float* res2 = theta + PM;                             // [p]
    int* ordp = reinterpret_cast<int*>(res2 + PM);        // [p]

    for (int e = tid; e < D * p; e += NT) Zb[e] = omega_entry((uint32_t)e);
    __syncthreads();

    int iters = 0;
    bool ok = true, have_vectors = false;
    mul_G<D, LD>(Gc, Zb, Yb, p, tid, NT);          // Y = G Omega
    __syncthreads();
    // Two attempts.  The power iteration stops when the block residual reaches the rounding
    // floor; the certification below then looks at each vector against its own gap.  If
    // only a residual is too large there, the second attempt takes the power iteration one
    // step further (Yb still holds G Z) and solves the Rayleigh-Ritz problem again; anything
    // else goes to the full route.  (Stopping earlier and retrying more often costs more than
    // it saves: a retry repeats the Jacobi solve.)
    for (int attempt = 0; attempt < 2; ++attempt) {
    if (attempt == 1) {
      ok = true;
      if (tid == 0) { s_why = 0; s_flags[0] = 0; s_flags[1] = 0; s_flags[2] = 0; }
      __syncthreads();
    }
    const float settle = tol.floor_rel;
    // force_iters > 0: exactly that many orthonormalised power steps (Algorithm 1 with
    // n_iter = force_iters - 1), no stopping rule and no retry
    const int max_it = force_iters > 0 ? min(force_iters, kMaxSubspaceIters) : kMaxSubspaceIters;
    for (int it = iters; it < max_it && ok; ++it) {
      // Cholesky-QR of the power step's Y = G Z:  A = Y^T Y = L L^T,  Z = Y L^-T
      mul_XtY<D, double, double>(Yb, Yb, Ad, p, LPD, tid, NT);
      __syncthreads();
      if (tid < 32) {
        const bool pd = cholesky_inverse_warp(Ad, Li, dref, p, LPD, lane);
        if (tid == 0) s_flags[3] = pd ? 0 : 1;
      }
      __syncthreads();
      if (s_flags[3]) { ok = false; if (tid == 0) s_why |= kWhyCholesky; break; }
      apply_Linv_t<D>(Yb, Li, Zb, p, LPD, tid, NT);
      __syncthreads();
      // next power step (kept in Yb), Rayleigh-Ritz matrix T = Z^T (G Z), block residual G Z - Z T
      mul_G<D, LD>(Gc, Zb, Yb, p, tid, NT);
      __syncthreads();
      mul_XtY<D, float, float>(Zb, Yb, Tc, p, LP, tid, NT);
      __syncthreads();
      iters = it + 1;
      if (it + 1 == max_it) break;
      // ||G Z - Z T||_F^2, accumulated per warp then by shared-memory atomics
      if (tid == 0) res2[0] = 0.f;
      __syncthreads();
      float part = 0.f;
      for (int t = tid; t < (D / 4) * p; t += NT) {
        const int j = t % p, i0 = (t / p) * 4;
        float zt[4];
        rows_dot_col<4>(Zb, Tc, p, LP, i0, j, zt);
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const float d = Yb[(i0 + m) * p + j] - zt[m];
          part = fmaf(d, d, part);
        }
      }
#pragma unroll
      for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      if (lane == 0) atomicAdd(&res2[0], part);
      __syncthreads();
      float tmax = 0.f;
      for (int k = 0; k < p; ++k) tmax = fmaxf(tmax, fabsf(Tc[k * LP + k]));
      const bool settled = sqrtf(res2[0]) <= settle * tmax;
      __syncthreads();
      // with oversampling (p > r) the extra directions never settle: two steps are the rule
      if (force_iters == 0 && (settled || (p > r && it >= 1))) break;
    }

    if (ok) {
      // symmetrise T into the planar block layout of the Jacobi, W = I
      const int hp = p >> 1;
      for (int e = tid; e < p * p; e += NT) {
        const int a = e / p, c = e % p;
        Wb[rblk_off(a, c, hp)] = (a == c) ? 1.f : 0.f;
        Tb[rblk_off(a, c, hp)] = 0.5f * (Tc[a * LP + c] + Tc[c * LP + a]);
      }
      __syncthreads();
      float tmax = 0.f;
      for (int k = 0; k < p; ++k) tmax = fmaxf(tmax, fabsf(Tb[rblk_off(k, k, hp)]));
      const int jt = min(NT, (hp * hp + 31) & ~31);
      if (tid < jt) {
        const int sw = ritz_jacobi(Tb, Wb, p, (kTolAbs * tmax) * (kTolAbs * tmax), stop2, s_flags, tid, jt);
        if (tid == 0) s_sweeps = sw;
      }
      __syncthreads();
      // the result sits in the buffer given by the parity of the rounds done; unpack it
      {
        const int sw = s_sweeps;
        const int fin = (((sw < 0 ? kMaxSweeps : sw) * (p - 1)) & 1) * rblk_size(hp);
        for (int e = tid; e < p * p; e += NT) {
          const int a = e / p, c = e % p;
          Wm[a * LP + c] = Wb[fin + rblk_off(a, c, hp)];
        }
        if (tid < p) { theta[tid] = Tb[fin + rblk_off(tid, tid, hp)]; res2[tid] = 0.f; }
      }
      __syncthreads();
      rank_descending(theta, ordp, p, tid);
      __syncthreads();

      pdl_trigger();     // the long part is over: the next kernel may start launching
      // Ritz vectors v = Z w and residuals G v - theta v of the r kept pairs
      for (int t = tid; t < (D / 2) * p; t += NT) {
        const int jr = t % p, i0 = (t / p) * 2;
        if (jr < r) {
          const int col = ordp[jr];
          float v[2], gv[2];
          rows_dot_col<2>(Zb, Wm, p, LP, i0, col, v);
          rows_dot_col<2>(Yb, Wm, p, LP, i0, col, gv);
          Xb[i0 * p + jr] = v[0];
          Xb[(i0 + 1) * p + jr] = v[1];
          const float th = theta[col];
          const float rho0 = gv[0] - th * v[0], rho1 = gv[1] - th * v[1];
          atomicAdd(&res2[jr], fmaf(rho0, rho0, rho1 * rho1));
        }
      }
      __syncthreads();

      // certification (see the file header); all quantities are of sc * G
      int good = 1;
      if (tid < r) {
        double kept = 0.0, rf2 = 0.0;
        for (int k = 0; k < r; ++k) { kept += (double)theta[ordp[k]]; rf2 += (double)res2[k]; }
        const float tail = (float)fmax((double)sc * s_trace - kept, 0.0);  // bounds every other eigenvalue
        const float th1 = theta[ordp[0]];
        const float thi = theta[ordp[tid]];
        const float thr_ = theta[ordp[r - 1]];
        const float cut = thr_ - tail - 2.f * sqrtf((float)rf2);
        float gap = (tid == r - 1) ? cut : thi - theta[ordp[tid + 1]];
        if (tid > 0) gap = fminf(gap, theta[ordp[tid - 1]] - thi);
        const float resn = sqrtf(res2[tid]);
        if (!(cut > 0.f)) atomicOr(&s_why, kWhyCut);
        if (!(thi > 0.f)) atomicOr(&s_why, kWhyNotPositive);
        if (!(resn <= fmaxf(tol.eps_vec * gap, tol.floor_rel * th1))) atomicOr(&s_why, kWhyResidual);
        good = (cut > 0.f) && (thi > 0.f) &&
               (resn <= fmaxf(tol.eps_vec * gap, tol.floor_rel * th1));
        if (!(resn == resn)) good = 0;
      }
      if (s_sweeps < 0) { good = 0; if (tid == 0) s_why |= kWhySweepCap; }   // Jacobi sweep cap reached
      ok = __syncthreads_and(good);
      have_vectors = true;
    }
    // retry only when a residual alone stood in the way and a power step is left
    if (ok || !have_vectors || s_why != kWhyResidual || iters >= kMaxSubspaceIters || force_iters > 0) break;
    __syncthreads();
    }   // attempts

    if (ok || (route == kRouteSubspace && have_vectors)) {
      // sign gauge and output
      float* sgn = res2;
      if (tid < r) {
        float best = -1.f, lead = 1.f;
        for (int j = 0; j < D; ++j) {
          const float v = Xb[j * p + tid];
          if (fabsf(v) > best) { best = fabsf(v); lead = v; }   // strict: lowest index wins a tie
        }
        S[(size_t)b * r + tid] = sqrtf(fmaxf(theta[ordp[tid]], 0.f) / sc);
        sgn[tid] = lead < 0.f ? -1.f : 1.f;
      }
      __syncthreads();
      for (int e = tid; e < D * r; e += NT) {
        const int j = e / r, i = e % r;
        V[(size_t)b * D * r + e] = Xb[j * p + i] * sgn[i];
      }
      if (tid == 0) {
        if (info) info[b] = ok ? 0 : SOLAR_INFO_NOT_CERTIFIED;
        if (route_taken) {
          const int sw = s_sweeps;
          route_taken[b] = kRouteSubspace | (iters << 8) | ((sw < 0 ? kMaxSweeps : sw) << 16) | (s_why << 24);
        }
      }
      return;
    }
    __syncthreads();
  }

  // ============================ route (2): full d x d Jacobi ============================
  full_jacobi_route<D, NT>(smem, s_flags, b, tid, r, sc, thr_abs2, stop2, s_why, sweep_cap, S, V, info,
                           route_taken);
}

template <int D>
cudaError_t launch_d(int B, int r, int p, int route, int sweep_cap, int force_iters, EigTol tol, const float* gpart,
                     const int* gram_status, int parts, int splits, float* S, float* V, int* info,
                     int* route_taken, cudaStream_t st) {
  using Cfg = EigCfg<D>;
  if (p > Cfg::PMAX) p = 0;
  cudaError_t e = cudaFuncSetAttribute(eig_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)Cfg::SMEM);
  if (e != cudaSuccess) return e;
  return launch_pdl(eig_kernel<D>, dim3(B), dim3(Cfg::THREADS), Cfg::SMEM, st, gpart, gram_status, parts, splits,
                    r, p, route, sweep_cap, force_iters, tol, S, V, info, route_taken);
}

}  // namespace

// Subspace dimension for rank r in width d: r rounded up to a multiple of 8 (a little
// oversampling; surplus directions of an exactly rank-r input deflate), if that is at most
// min(32, d/2); otherwise 0: the subspace route brings nothing.
int eig_subspace_dim(int d, int r) {
  const int p = (r + 7) / 8 * 8;
  return (p <= 32 && 2 * p <= d) ? p : 0;
}

cudaError_t launch_eig(int B, int d, int r, solar_dtype_t dt, int route, int sweep_cap, int force_iters,
                       const float* gpart, const int* gram_status, int parts, int splits, float* gsum, float* S,
                       float* V, int* info, int* route_taken, cudaStream_t st) {
  if (sweep_cap <= 0 || sweep_cap > kMaxSweeps) sweep_cap = kMaxSweeps;
  // AUTO and TRIDIAG: the tridiagonal route (with the Jacobi solve behind it in AUTO)
  if (route == SOLAR_ROUTE_AUTO || route == SOLAR_ROUTE_TRIDIAG)
    return launch_eig_tridiag(B, d, r, dt, route, sweep_cap, gpart, gram_status, parts, splits, gsum, S, V, info,
                              route_taken, nullptr, st);
  EigTol tol;
  if (dt == SOLAR_BF16) {
    tol.eps_vec = 1e-3f; tol.floor_rel = 256.f * kUnit; tol.sweep_stop = 1e-3f;
  } else {
    tol.eps_vec = 1e-5f; tol.floor_rel = 32.f * kUnit; tol.sweep_stop = 1e-5f;
  }
  const int p = eig_subspace_dim(d, r);
  switch (d) {
    case 32: return launch_d<32>(B, r, p, route, sweep_cap, force_iters, tol, gpart, gram_status, parts, splits, S, V, info, route_taken, st);
    case 64: return launch_d<64>(B, r, p, route, sweep_cap, force_iters, tol, gpart, gram_status, parts, splits, S, V, info, route_taken, st);
    case 128: return launch_d<128>(B, r, p, route, sweep_cap, force_iters, tol, gpart, gram_status, parts, splits, S, V, info, route_taken, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace solar
