// Parallel two-sided Jacobi on a whole d x d symmetric matrix in shared memory -- the
// eigensolver that is valid for any spectrum (Eq. 9's exact truncated SVD) -- and the small
// pieces it shares with the other routes.  Included by the eigensolver kernels only.
//
// Round-robin tournament in systolic form: the matrix is indexed by slot, the pairs of every
// round are the slots (2i, 2i+1), and a fixed slot move after each round makes every two
// indices meet once in n-1 rounds.  In one round every 2x2 block is touched by exactly one
// thread, which applies the row pair's rotation from the left and the column pair's from the
// right; the matrix is double-buffered, so a round costs ONE barrier.  The 2x2 blocks are
// stored in four planes so that the accesses of a warp are (nearly) free of bank conflicts.
#pragma once

#include <math.h>

#include "solar_internal.cuh"

namespace solar {

constexpr float kTolRel = 2.3841858e-07f;  // 2^-22: |g_pq| <= tol*sqrt(g_pp g_qq) counts as zero
constexpr float kTolAbs = 7.4505806e-09f;  // 2^-27 of the largest diagonal entry
constexpr float kUnit = 5.9604645e-08f;    // 2^-24, fp32 unit roundoff

// route_taken[b] = route | detail << 8 | sweeps or passes << 16 | kWhy* bits << 24
constexpr int kRouteSubspace = 1, kRouteFull = 2, kRouteTridiag = 3;
// Why a route's result was not certified (0 = it was, or it was not tried):
constexpr int kWhyCut = 1;          // the trace bound does not separate theta_r from the rest
constexpr int kWhyResidual = 2;     // a residual is too large for its gap
constexpr int kWhyNotPositive = 4;  // a kept Ritz value is not positive (rank(H) < r)
constexpr int kWhySweepCap = 8;     // the Ritz Jacobi hit its sweep cap
constexpr int kWhyCholesky = 16;    // non-finite pivot in the Cholesky-QR
constexpr int kWhyOrtho = 32;       // tridiagonal route: vectors of a cluster came out dependent
constexpr int kWhyTrace = 64;       // tridiagonal route: trace of T differs from trace of G, or not finite
constexpr int kWhyGap = 128;        // tridiagonal route: a gap between kept eigenvalues is too small for its accuracy

// Rotation J = [[c, s], [-s, c]] that annihilates g_pq of the 2x2 symmetric block
// [[a, g], [g, b]]; identity when g is negligible (or not a number).  Returned
// as s, tau = s/(1+c) and t = s/c: columns are updated in the cancellation-free
// form x_p' = x_p - s (x_q + tau x_p), x_q' = x_q + s (x_p - tau x_q), and the
// diagonal as a' = a - t g, b' = b + t g, so a near-identity rotation perturbs
// the matrix by O(s) instead of by a rounding error of the full entry.
// `big` is set when the rotated pair had g^2 > stop2 |a b|.  The matrix is scaled so
// that its largest diagonal entry lies in [1, 2): squares cannot overflow, and entries
// whose squares underflow are below the absolute threshold.  The approximate rsqrt
// (2 ulp) only moves the rotation angle by a rounding error.
struct Rot { float s, tau, t; };

__device__ __forceinline__ Rot jacobi_rot(float a, float b, float g, float thr_abs2, float stop2,
                                          bool& big) {
  const float g2 = g * g;
  const float ab = fabsf(a * b);
  const bool act = (g2 > thr_abs2) && (g2 > (kTolRel * kTolRel) * ab);
  big = act && (g2 > stop2 * ab);
  // With d = b - a and h = sqrt(d^2 + 4 g^2):  cos^2 = (h + |d|) / (2 h),
  // sin = sgn(d) g / (h cos),  tan = sin / cos,  tau = sin / (1 + cos).
  // Two dependent special-function evaluations (both rsqrt); 1 / (1 + cos), with
  // 1 + cos in [1.707, 2], comes from a linear guess and two Newton steps.
  const float dlt = b - a;
  const float rh = rsqrtf(fmaf(dlt, dlt, 4.f * g2));
  const float c2 = fmaf(0.5f * fabsf(dlt), rh, 0.5f);
  const float rc = rsqrtf(c2);
  const float c = c2 * rc;
  const float s = copysignf(g * rh, dlt * g) * rc;
  const float t = s * rc;
  const float u = 1.f + c;
  float y = fmaf(-0.29289f, u, 1.08579f);
  y = y * fmaf(-u, y, 2.f);
  y = y * fmaf(-u, y, 2.f);
  Rot r;
  r.s = act ? s : 0.f;
  r.t = act ? t : 0.f;
  r.tau = act ? s * y : 0.f;
  return r;
}

__device__ __forceinline__ void rot_apply(const Rot& r, float& xp, float& xq) {
  const float p = xp, q = xq;
  xp = fmaf(-r.s, fmaf(r.tau, p, q), p);
  xq = fmaf(r.s, fmaf(-r.tau, q, p), q);
}

// Barrier among the first `nthreads` threads of the CTA (a multiple of 32).
__device__ __forceinline__ void bar_named(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Slot move of the tournament: slot 0 stays; slot 1 -> 2; slot 2i -> 2i+2 (1 <= i <= p/2-2);
// slot p-2 -> p-1; slot 2i+1 -> 2i-1 (i >= 1).  Nothing has to track which original index
// sits in a slot: eigenvalue and eigenvector simply travel together.
__device__ __forceinline__ int slot_next(int u, int p) {
  if (u == 0) return 0;
  if (u == 1) return 2;
  if (u & 1) return u - 2;
  return (u == p - 2) ? p - 1 : u + 2;
}
// Offset (in floats) of element (u, v) in the planar 2x2-block layout of the full route: block
// (u/2, v/2), whose four entries sit in four planes [2*(u%2) + v%2][u/2][v/2] with row pitch
// p/2 + 1.
__device__ __forceinline__ int blk_off(int u, int v, int hp) {
  return (((u & 1) << 1) + (v & 1)) * (hp * (hp + 1)) + (u >> 1) * (hp + 1) + (v >> 1);
}

// Ranks of lam[0..n) in descending order (ties: lower index first): order[rank] = index.
__device__ __forceinline__ void rank_descending(const float* lam, int* order, int n, int tid) {
  if (tid < n) {
    const float li = lam[tid];
    int rank = 0;
    for (int j = 0; j < n; ++j) {
      const float lj = lam[j];
      rank += (lj > li) || (lj == li && j < tid);
    }
    order[rank] = tid;
  }
}

// Floats of shared memory the full route needs: the current and the next matrix, the
// eigenvector matrix ([D][D + 4] each), lam[D], order[D], perm[2][D].
template <int D> constexpr int full_jacobi_floats() { return 3 * D * (D + 4) + 4 * D; }

// The full route on the CTA's NT threads.  On entry smem[0 .. D*(D+4)) holds sc*G row-major
// with row pitch D + 4 (sc the power of two that brings the largest diagonal entry into
// [1, 2)); every thread of the CTA calls this.  T is kept in the planar block layout,
// double-buffered (buffer 0 overlays the row-major G, buffer 1 the next matrix slot); the
// eigenvector matrix W stays COLUMN-major and in place: slot v's vector is column perm[v], the
// slot move only permutes `perm`.  Lanes run along the row blocks I, so a warp reads one W
// column pair as 32 consecutive 8-byte pieces, the column rotation (and its perm lookup) is
// uniform across the warp, and every T access is conflict-free.  Thread (I, Jb) owns the
// blocks (I, Jb + c*NJ), c < PTJ.  At most sweep_cap (<= kMaxSweeps) sweeps are made; a user that
// has not converged by then is flagged SOLAR_INFO_NOT_CONVERGED.  Writes S, V, info and
// route_taken of user b.
template <int D, int NT>
__device__ __forceinline__ void full_jacobi_route(float* smem, int* s_flags, int b, int tid, int r,
                                                  float sc, float thr_abs2, float stop2, int why,
                                                  int sweep_cap, float* __restrict__ S, float* __restrict__ V,
                                                  int* __restrict__ info, int* __restrict__ route_taken) {
  constexpr int LD = D + 4;
  float* Gc = smem;                 // current matrix
  float* Gn = smem + D * LD;        // next matrix
  float* Vm = smem + 2 * D * LD;    // accumulated rotations (eigenvectors in columns)
  float* lam = smem + 3 * D * LD;   // [D] eigenvalues
  int* order = reinterpret_cast<int*>(lam + D);   // [D] column holding the k-th largest eigenvalue
  const int lane = tid & 31;
  // For d = 64 the four planes lie one word further apart than HP * (HP + 1): counted over every
  // access of a round that leaves 9 % extra wavefronts from bank conflicts instead of 54 %;
  // for d = 128 the same offset measured slower.
  constexpr int HP = D / 2, NJ = NT / HP, PTJ = HP / NJ, XP = (HP == 32) ? 1 : 0;
  constexpr int PLN = HP * (HP + 1) + XP, TBS = 4 * PLN;
  static_assert(NT % HP == 0 && HP % NJ == 0 && TBS <= D * LD && D * D <= D * LD, "full-route tiling");
  static_assert(HP == 16 || HP == 32 || HP == 64, "rotation sharing by shuffle");
  float* Wc = Vm;                                  // [D cols][D rows]
  int* perm = order + D;                           // [2][D]
  const int I = tid % HP, Jb = tid / HP;

  float xin[PTJ][4];
#pragma unroll
  for (int c = 0; c < PTJ; ++c) {
    const int J = Jb + c * NJ;
    xin[c][0] = Gc[(2 * I) * LD + 2 * J];     xin[c][1] = Gc[(2 * I) * LD + 2 * J + 1];
    xin[c][2] = Gc[(2 * I + 1) * LD + 2 * J]; xin[c][3] = Gc[(2 * I + 1) * LD + 2 * J + 1];
  }
  __syncthreads();                                 // all of row-major G is in registers
  int tdst[PTJ][4];
  const int r0 = slot_next(2 * I, D), r1 = slot_next(2 * I + 1, D);
#pragma unroll
  for (int c = 0; c < PTJ; ++c) {
    const int J = Jb + c * NJ, src = I * (HP + 1) + J;
#pragma unroll
    for (int q = 0; q < 4; ++q) Gc[q * PLN + src] = xin[c][q];
    const int c0 = slot_next(2 * J, D), c1 = slot_next(2 * J + 1, D);
    tdst[c][0] = blk_off(r0, c0, HP) + XP * (((r0 & 1) << 1) + (c0 & 1));
    tdst[c][1] = blk_off(r0, c1, HP) + XP * (((r0 & 1) << 1) + (c1 & 1));
    tdst[c][2] = blk_off(r1, c0, HP) + XP * (((r1 & 1) << 1) + (c0 & 1));
    tdst[c][3] = blk_off(r1, c1, HP) + XP * (((r1 & 1) << 1) + (c1 & 1));
  }
  for (int e = tid; e < D * D; e += NT) Wc[e] = (e / D == e % D) ? 1.f : 0.f;
  if (tid < D) perm[tid] = tid;
  if (tid < 3) s_flags[tid] = 0;
  __syncthreads();

  const int cap = min(max(sweep_cap, 1), kMaxSweeps);
  int converged = 0, sweeps_done = cap, cur = 0;
  for (int sweep = 0; sweep < cap; ++sweep) {
    if (tid == 0) s_flags[(sweep + 1) % 3] = 0;
    bool worst = false;
    for (int k = 0; k < D - 1; ++k) {
      const float* Tc = cur ? Gn : Gc;
      float* Tn = cur ? Gc : Gn;
      const int* pc = perm + cur * D;
      // The lanes of every warp compute the round's HP rotations between them (lane l takes
      // the pairs l, l + 32, ...); a thread's row rotation is among its own, and the column
      // rotations, uniform across the warp, come by shuffle -- instead of every thread
      // computing one rotation per block it owns.
      constexpr int NR = (HP + 31) / 32;
      Rot rl[NR];
#pragma unroll
      for (int q = 0; q < NR; ++q) {
        const int pr = (HP >= 32) ? q * 32 + lane : lane % HP;
        const int sp = pr * (HP + 1) + pr;
        bool big;
        rl[q] = jacobi_rot(Tc[sp], Tc[3 * PLN + sp], Tc[PLN + sp], thr_abs2, stop2, big);
        worst |= big;
      }
      Rot rr = rl[0];
      if (NR == 2 && I >= 32) rr = rl[NR - 1];
#pragma unroll
      for (int c = 0; c < PTJ; ++c) {
        const int J = Jb + c * NJ, src = I * (HP + 1) + J;
        const Rot& rs = (NR == 2 && J >= 32) ? rl[NR - 1] : rl[0];   // J is uniform across the warp
        Rot rc;
        rc.s = __shfl_sync(0xffffffffu, rs.s, J & 31);
        rc.tau = __shfl_sync(0xffffffffu, rs.tau, J & 31);
        rc.t = rr.t;                       // used only where I == J
        float x00 = Tc[src], x01 = Tc[PLN + src], x10 = Tc[2 * PLN + src], x11 = Tc[3 * PLN + src];
        float2* wa = reinterpret_cast<float2*>(Wc + pc[2 * J] * D + 2 * I);
        float2* wb = reinterpret_cast<float2*>(Wc + pc[2 * J + 1] * D + 2 * I);
        float2 va = *wa, vb = *wb;
        if (I == J) {                      // the pair's own diagonal block
          const float tg = rc.t * x01;
          x00 -= tg; x11 += tg;
          if (rc.s != 0.f) { x01 = 0.f; x10 = 0.f; }
        } else {
          rot_apply(rc, x00, x01); rot_apply(rc, x10, x11);   // columns
          rot_apply(rr, x00, x10); rot_apply(rr, x01, x11);   // rows
        }
        rot_apply(rc, va.x, vb.x); rot_apply(rc, va.y, vb.y);
        Tn[tdst[c][0]] = x00; Tn[tdst[c][1]] = x01; Tn[tdst[c][2]] = x10; Tn[tdst[c][3]] = x11;
        *wa = va; *wb = vb;
      }
      if (tid < D) perm[(cur ^ 1) * D + slot_next(tid, D)] = pc[tid];
      if (k == D - 2 && worst) s_flags[sweep % 3] = 1;
      __syncthreads();
      cur ^= 1;
    }
    if (s_flags[sweep % 3] == 0) { converged = 1; sweeps_done = sweep + 1; break; }
  }

  // ---- order the eigenvalues, keep r, fix the sign of each vector ----------------
  const float* Tf = cur ? Gn : Gc;
  const int* pf = perm + cur * D;
  if (tid < D) lam[tid] = Tf[(tid & 1) * 3 * PLN + (tid >> 1) * (HP + 1) + (tid >> 1)];
  __syncthreads();
  rank_descending(lam, order, D, tid);
  __syncthreads();
  float* sgn = cur ? Gc : Gn;   // reuse: [r] signs
  if (tid < r) {
    const float* col = Wc + pf[order[tid]] * D;
    float best = -1.f, lead = 1.f;
    for (int j = 0; j < D; ++j) {
      const float v = col[j];
      if (fabsf(v) > best) { best = fabsf(v); lead = v; }   // strict: lowest index wins a tie
    }
    sgn[tid] = lead < 0.f ? -1.f : 1.f;
    S[(size_t)b * r + tid] = sqrtf(fmaxf(lam[order[tid]], 0.f) / sc);
  }
  __syncthreads();
  for (int e = tid; e < D * r; e += NT) {
    const int j = e / r, i = e % r;
    V[(size_t)b * D * r + e] = Wc[pf[order[i]] * D + j] * sgn[i];
  }
  if (tid == 0) {
    if (info) info[b] = converged ? 0 : SOLAR_INFO_NOT_CONVERGED;
    if (route_taken) route_taken[b] = kRouteFull | (sweeps_done << 16) | (why << 24);
  }
}

}  // namespace solar
