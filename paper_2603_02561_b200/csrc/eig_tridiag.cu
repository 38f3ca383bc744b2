// Batched symmetric eigensolver, tridiagonal route: the top-r eigenpairs of every Gram matrix
// G_b = H_b^T H_b (Eq. 9 without U: s_i = sqrt(lambda_i), V = eigenvectors) by the classical
// dense-symmetric chain, one CTA per user, sized so that a user costs tens of thousands of warp
// instructions and a modest register and shared-memory footprint (several CTAs share an SM with
// the streaming kernels of other requests) instead of the hundreds of thousands of a Jacobi solve:
//
//   1. G = sum of the slices' partial Grams (fixed order), scaled by a power of two.
//   2. Householder tridiagonalisation T = Q^T G Q with the matrix held in REGISTERS, spread over
//      all warps of the CTA: thread (warp w, lane l) owns rows l, l+32, ... and the columns of
//      its warp's 4-column groups, so the symmetric matrix-vector product and the rank-2 update
//      of a step are FMAs on statically indexed registers.  Every warp computes the step's
//      scalars redundantly (column norm and p^T v by shuffles); the warps exchange only their
//      partial products, through shared memory, at ONE barrier per step.  The next step's
//      column comes from the owner of row k+1 (by symmetry) before the update and is corrected
//      by the rank-2 term, so no step waits for the update of the one before.
//   3. The r largest eigenvalues of T by multisection on Sturm counts: one lane per eigenvalue,
//      one interior point per warp and step (4 or 8 points), the counts taken from the
//      three-term recurrence of the leading principal minors with a power-of-two rescale every
//      four steps -- one FMA per step on the dependency chain instead of a division.
//   4. One eigenvector per eigenvalue from the twisted factorisation of T - lambda I (forward
//      and backward pivot sequences as ratios of consecutive minors, twist at the smallest
//      |gamma_k|): inverse iteration from the best unit vector, O(d) per vector, no pivoting.
//   5. Back-transformation V = Q Z: four threads per vector, each applying the d-2 reflectors to
//      its quarter of the rows held in registers.
//   6. Gram-Schmidt passes in matrix form, V <- V (I - strict_upper(V^T V - I)) D^-1, repeated
//      while V^T V - I is above the rounding level (vectors of close eigenvalues come out of
//      step 4 with a mutual error of order eps |T| / gap); a column is only ever corrected by
//      the columns of larger eigenvalues.
//   7. Rayleigh quotients theta_i = v_i^T G v_i and residuals G v_i - theta_i v_i against the
//      ORIGINAL G: the result is accepted only if every residual is small against its gap (or
//      at the rounding floor), V^T V = I to rounding, and trace(T) = trace(G); otherwise the
//      CTA runs the parallel Jacobi eigensolver on the whole matrix, which is valid for any
//      spectrum (clusters of equal eigenvalues, rank(H) < r, ...).
//
// A warp that runs alone on its scheduler pays the full latency of every branch and of every
// dependent instruction; the code below is therefore straight-line over static ranges (the
// Householder loop is cut into stages with fixed live rows and columns), keeps divisions off
// the dependency chains, and spreads independent work over the warps.
#include "eig_jacobi.cuh"
#include "project_mma.cuh"

namespace solar {

namespace {

constexpr unsigned kFull = 0xffffffffu;

template <int D> struct TriCfg {
  static constexpr int NT = (D == 128) ? 256 : 128;   // threads of the CTA
  static constexpr int NW = NT / 32;
  static constexpr int RPT = D / 32;                  // rows per thread: l + 32 q
  static constexpr int CPT = D / NW;                  // columns per thread ...
  static constexpr int NG = CPT / 4;                  // ... as 4-column groups: group g of warp w = columns 4 (w + NW g) ..+3
  static constexpr int SS = 4 * NW;                   // steps per stage: from step s * SS on, the groups g < s are finished
  static constexpr int LD = D + 4;                    // pitch of the staged row-major G
  static constexpr int NB = D / 4;                    // 4-column blocks of a row
  static_assert(SS * NG == D && RPT * 32 == D, "ownership covers the matrix");
};

// Shared-memory layout (floats) for subspace width RP = 32 * ceil(r / 32).
template <int D, int RP> struct TriSmem {
  using C = TriCfg<D>;
  static constexpr int HV = 0;                                   // [D][D] reflector k in row k; later G
  static constexpr int VS = HV + D * D;                          // [D][RP] V
  static constexpr int WORK_FLOATS = (D * C::LD > 2 * D * RP) ? D * C::LD : 2 * D * RP;
  static constexpr int WORK = VS + D * RP;                       // staged G | tf, tb [D][RP] | V'
  static constexpr int EM = WORK + WORK_FLOATS;                  // [RP][RP] V^T V - I (before: multisection flags)
  static constexpr int DG = EM + RP * RP;                        // [D] diagonal of T
  static constexpr int EO = DG + D;                              // [D] off-diagonal: e[k] couples k, k+1
  static constexpr int E2 = EO + D;                              // [D] e2s[i] = e[i-1]^2 (floored), e2s[0] = 0
  static constexpr int BE = E2 + D;                              // [D] beta of reflector k
  static constexpr int XP = BE + D;                              // [2][D] row k+1 before the update of step k
  static constexpr int TP = XP + 2 * D;                          // [2][NW][D] the warps' partial products A v
  static constexpr int PV = TP + 2 * C::NW * D;                  // [2][8] the warps' partial p^T v
  static constexpr int LAM = PV + 16;                            // [RP] eigenvalues of T
  static constexpr int TH = LAM + RP;                            // [RP] Rayleigh quotients
  static constexpr int RH = TH + RP;                             // [RP] squared residual norms
  static constexpr int SG = RH + RP;                             // [RP] gauge signs; before: 1 / |z|
  static constexpr int KT = SG + RP;                             // [RP] twist index (int)
  static constexpr int PART = KT + RP;                           // [2][NW][RP] per-warp partial results
  static constexpr int TRI_FLOATS = PART + 2 * C::NW * RP;
  // the projection epilogue: V Sigma, Key_r^T, two weights (FFMA form) or the tensor-core form's staging
  static constexpr int EPI_FFMA = 2 * D * RP + 2 * D * D;
  static constexpr int EPI_MMA = (D >= 64) ? pmma::Lay<(D >= 64 ? D : 64)>::bytes(RP) / 4 : 0;
  static constexpr int EPI_FLOATS = EPI_FFMA > EPI_MMA ? EPI_FFMA : EPI_MMA;
  static constexpr int M1 = TRI_FLOATS > full_jacobi_floats<D>() ? TRI_FLOATS : full_jacobi_floats<D>();
  static constexpr int FLOATS = M1 > EPI_FLOATS ? M1 : EPI_FLOATS;
  static constexpr size_t BYTES = (size_t)FLOATS * sizeof(float);
  static_assert(DG % 4 == 0 && EO % 4 == 0 && E2 % 4 == 0 && XP % 4 == 0 && TP % 4 == 0 && PV % 4 == 0 &&
                EM % 4 == 0 && WORK % 4 == 0 && VS % 4 == 0, "16-byte alignment of the regions");
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
  return v;
}
// 16-byte store to shared memory under a predicate, without a branch.
__device__ __forceinline__ void sts_v4_if(float* p, float a, float b, float c, float d, bool pred) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.s32 p, %5, 0;\n\t@p st.shared.v4.f32 [%0], {%1, %2, %3, %4};\n\t}"
               ::"r"((uint32_t)__cvta_generic_to_shared(p)), "f"(a), "f"(b), "f"(c), "f"(d), "r"((int)pred)
               : "memory");
}
// 1 / sqrt(x) and 1 / x to fp32 accuracy (approximation plus one Newton step): the reflector
// I - beta v v^T is orthogonal only as far as beta v^T v = 2 holds.
__device__ __forceinline__ float rsqrt_acc(float x) {
  const float y = rsqrtf(x);
  return y * fmaf(-0.5f * x * y, y, 1.5f);
}
__device__ __forceinline__ float rcp_acc(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y * fmaf(-x, y, 2.f);
}

// ---- Householder steps of stage S: k in [S * SS, min((S + 1) * SS, D - 2)) -------------------
// From step S * SS on the column groups g < S and the row slots q < Q0 are finished, so every
// range below is static.  State carried from step to step: the matrix a, and column k of the
// current matrix at the thread's rows (xr) and columns (xc; by symmetry row k).
template <int D, int S>
__device__ __forceinline__ void tri_stage(float (&a)[TriCfg<D>::RPT][TriCfg<D>::CPT], float (&xr)[TriCfg<D>::RPT],
                                          float (&xc)[TriCfg<D>::CPT], float* __restrict__ hv,
                                          float* __restrict__ xpre, float* __restrict__ tpart,
                                          float* __restrict__ pvp, float* __restrict__ dg, float* __restrict__ eo,
                                          float* __restrict__ betas, int tid, float& tr_rest, float& tr_comp, float stop_tr,
                                          float stop_x2, int r, int& k_stop) {
  using C = TriCfg<D>;
  constexpr int NW = C::NW, RPT = C::RPT, NG = C::NG, SS = C::SS;
  constexpr int G0 = S;                                               // first live column group
  constexpr int Q0 = (S * SS >= 31) ? (S * SS - 31) / 32 + 1 : 0;     // first live row slot
  constexpr int K1 = ((S + 1) * SS < D - 2) ? (S + 1) * SS : D - 2;
  const int lane = tid & 31, warp = tid >> 5;
  if (k_stop >= 0) return;
#pragma unroll 1
  for (int k = S * SS; k < K1; ++k) {
    const int k1 = k + 1, par = k & 1, q1 = k1 >> 5, l1 = k1 & 31;
    // row k+1 of the current matrix at my columns, for the next step's vector (no branch: the
    // store is predicated; one lane per warp owns the row)
#pragma unroll
    for (int q = Q0; q < RPT; ++q)
#pragma unroll
      for (int g = G0; g < NG; ++g)
        sts_v4_if(xpre + par * D + 4 * (warp + NW * g), a[q][4 * g], a[q][4 * g + 1], a[q][4 * g + 2],
                  a[q][4 * g + 3], q == q1 && lane == l1);
    // x = column k below the subdiagonal; its norm; alpha, beta, v
    float xs[RPT], sq = 0.f, c1 = xr[RPT - 1], ck = xr[RPT - 1];
#pragma unroll
    for (int q = RPT - 1; q >= 0; --q) {
      xs[q] = (q >= Q0 && lane + 32 * q > k1) ? xr[q] : 0.f;
      sq = fmaf(xs[q], xs[q], sq);
      c1 = (q == q1) ? xr[q] : c1;
      ck = (q == (k >> 5)) ? xr[q] : ck;
    }
    const float x1 = __shfl_sync(kFull, c1, l1), dk = __shfl_sync(kFull, ck, k & 31);
    const float tail2 = warp_sum(sq);
    // With nothing to annihilate (an exactly zero tail) the reflector is the identity: beta = 0
    // makes p, w and the update vanish, and the step still hands on column k+1.
    const bool reflect = tail2 > 1e-35f;
    const float s2 = fmaf(x1, x1, tail2);
    // Rank-revealing stop: once the rows below k carry a negligible trace (G is positive
    // semi-definite, so that bounds every entry of the block) and row k hardly couples to them,
    // T ends at row k.  A history of low rank -- the premise of the method -- then costs its rank
    // in Householder steps, and every later phase works on the shorter T.
    {                                    // tr_rest -= dk, compensated (the trace is ~10^7 stop thresholds)
      const float y = -dk - tr_comp, t = tr_rest + y;
      tr_comp = (t - tr_rest) - y;
      tr_rest = t;
    }
    if (k1 >= r && tr_rest <= stop_tr && s2 <= stop_x2) {
      if (tid == 0) { dg[k] = dk; eo[k] = 0.f; betas[k] = 0.f; }
      k_stop = k;
      return;
    }
    const float nrm = s2 * rsqrt_acc(fmaxf(s2, 1e-37f));
    const float alpha = reflect ? -copysignf(nrm, x1) : x1;
    const float vk1 = reflect ? x1 - alpha : 0.f;
    const float beta = reflect ? rcp_acc(nrm * fabsf(vk1)) : 0.f;
    if (tid == 0) { dg[k] = dk; eo[k] = alpha; betas[k] = beta; }
    float vr[RPT], vc[NG][4];
#pragma unroll
    for (int q = Q0; q < RPT; ++q) {
      vr[q] = (lane + 32 * q == k1) ? vk1 : xs[q];
      if (warp == 0) hv[k * D + lane + 32 * q] = vr[q];        // reflector k (rows <= k stay zero)
    }
#pragma unroll
    for (int g = G0; g < NG; ++g)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int col = 4 * (warp + NW * g) + c;
        vc[g][c] = (col == k1) ? vk1 : (col > k1 ? xc[4 * g + c] : 0.f);
      }
    // my columns' share of A v at my rows, and of p^T v
    float dp = 0.f;
#pragma unroll
    for (int q = Q0; q < RPT; ++q) {
      float t0 = 0.f, t1 = 0.f;
#pragma unroll
      for (int g = G0; g < NG; ++g) {
        t0 = fmaf(a[q][4 * g], vc[g][0], t0);     t1 = fmaf(a[q][4 * g + 1], vc[g][1], t1);
        t0 = fmaf(a[q][4 * g + 2], vc[g][2], t0); t1 = fmaf(a[q][4 * g + 3], vc[g][3], t1);
      }
      const float pq = t0 + t1;
      tpart[(par * NW + warp) * D + lane + 32 * q] = pq;
      dp = fmaf(pq, vr[q], dp);
    }
    dp = warp_sum(dp);
    if (lane == 0) pvp[par * 8 + warp] = dp;
    __syncthreads();
    // p = beta A v at my rows, my columns and at k+1; K = beta p^T v / 2; w = p - K v
    float pvs = 0.f, pk1 = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) { pvs += pvp[par * 8 + w]; pk1 += tpart[(par * NW + w) * D + k1]; }
    const float kk = 0.5f * beta * beta * pvs;
    const float wk1 = fmaf(-kk, vk1, beta * pk1);
    float wr[RPT], wc[NG][4], prow[RPT];
#pragma unroll
    for (int q = 0; q < RPT; ++q) prow[q] = 0.f;
#pragma unroll
    for (int q = Q0; q < RPT; ++q) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) t += tpart[(par * NW + w) * D + lane + 32 * q];
      prow[q] = t;
      wr[q] = (lane + 32 * q > k) ? fmaf(-kk, vr[q], beta * t) : 0.f;
      // column k+1 of the updated matrix at my rows: row k+1 before the update, corrected
      xr[q] = fmaf(-wr[q], vk1, fmaf(-vr[q], wk1, xpre[par * D + lane + 32 * q]));
    }
#pragma unroll
    for (int g = G0; g < NG; ++g) {
      const int cb = 4 * (warp + NW * g);
      const float4 xp = *reinterpret_cast<const float4*>(xpre + par * D + cb);
      const float xx[4] = {xp.x, xp.y, xp.z, xp.w};
      float tt[4];
      // (A v) at column cb + c is the row sum held by the lane that owns row cb + c (slot
      // 4 NW g / 32 of that lane): one shuffle instead of NW loads and adds
#pragma unroll
      for (int c = 0; c < 4; ++c) tt[c] = __shfl_sync(kFull, prow[(4 * NW * g) >> 5], (cb + c) & 31);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        wc[g][c] = (cb + c > k) ? fmaf(-kk, vc[g][c], beta * tt[c]) : 0.f;
        xc[4 * g + c] = fmaf(-wc[g][c], vk1, fmaf(-vc[g][c], wk1, xx[c]));
      }
    }
    // A <- A - v w^T - w v^T on the live block
#pragma unroll
    for (int q = Q0; q < RPT; ++q)
#pragma unroll
      for (int g = G0; g < NG; ++g)
#pragma unroll
        for (int c = 0; c < 4; ++c)
          a[q][4 * g + c] = fmaf(-vr[q], wc[g][c], fmaf(-wr[q], vc[g][c], a[q][4 * g + c]));
  }
}

// Number of eigenvalues of T below x, for CH values of x at once.  p_{i+1} = (d_i - x) p_i -
// e_{i-1}^2 p_{i-1} is the leading principal minor of order i+1 of T - x I; the sign changes
// along p_0 = 1, p_1, ..., p_D count the eigenvalues below x.  The off-diagonal squares are
// floored above zero, so an exact zero never persists, and an isolated zero gives one change
// whichever sign the hardware gives it.
template <int D, int CH>
__device__ __forceinline__ void sturm(const float* __restrict__ dg, const float* __restrict__ e2s,
                                      const float (&x)[CH], int (&cnt)[CH], int nb4) {
  float p[CH], q[CH];
  unsigned n[CH];
#pragma unroll
  for (int h = 0; h < CH; ++h) { p[h] = 1.f; q[h] = 0.f; n[h] = 0; }
#pragma unroll 4
  for (int ib = 0; ib < nb4; ++ib) {
    const float4 d4 = *reinterpret_cast<const float4*>(dg + 4 * ib);
    const float4 e4 = *reinterpret_cast<const float4*>(e2s + 4 * ib);
    const float dd[4] = {d4.x, d4.y, d4.z, d4.w}, ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int h = 0; h < CH; ++h) {
        const float t = ee[u] * q[h];
        const float rr = fmaf(dd[u] - x[h], p[h], -t);
        n[h] += (__float_as_uint(rr) ^ __float_as_uint(p[h])) >> 31;
        q[h] = p[h]; p[h] = rr;
      }
    // bring the larger of (p, q) back into [1, 2): |d - x| and e^2 are bounded by the scaling of G,
    // so four steps can neither overflow nor (factors above 2^-23 each) underflow
#pragma unroll
    for (int h = 0; h < CH; ++h) {
      const unsigned m = __float_as_uint(fmaxf(fabsf(p[h]), fabsf(q[h]))) >> 23;
      const float sc = __uint_as_float((254u - m) << 23);
      p[h] *= sc; q[h] *= sc;
    }
  }
#pragma unroll
  for (int h = 0; h < CH; ++h) cnt[h] = (int)n[h];
}

// Acceptance thresholds (chosen by the storage type).
struct TriTol {
  float eps_vec;     // bound on sin(angle) of a kept vector implied by its residual and gap
  float floor_rel;   // residuals below floor_rel * theta_1 are at the rounding level of fp32
  float ortho;       // largest |V^T V - I| entry that needs no further orthogonalisation
  float gap_min;     // smallest gap between kept eigenvalues, relative to the largest, the route is trusted with
  float stop_trace;  // the reduction stops once the remaining rows' trace is below this fraction of trace(G) ...
  float stop_couple; // ... and the current row couples to them by less than this fraction of it
  float sweep_stop;  // of the Jacobi fallback
};

// The eigensolve of user blockIdx.x; every thread of the CTA calls it and all leave together.
// With want_vs, a certified tridiagonal result also leaves V Sigma at the start of the dynamic
// shared memory ([D][rp], rp = r rounded up to 4, zero in the padding) and true is returned.
template <int D, int RP>
__device__ __forceinline__ bool eig_user(const float* __restrict__ gpart, const int* __restrict__ gram_status,
                                         int parts, int splits, float* __restrict__ gsum, int r, int route, int sweep_cap,
                                         const TriTol& tol, bool want_vs, bool late_trigger, float* __restrict__ S,
                                         float* __restrict__ V, int* __restrict__ info,
                                         int* __restrict__ route_taken) {
  using Cfg = TriCfg<D>;
  using L = TriSmem<D, RP>;
  constexpr int NT = Cfg::NT, NW = Cfg::NW, RPT = Cfg::RPT, CPT = Cfg::CPT, NG = Cfg::NG, LD = Cfg::LD;
  constexpr int NE = RP / 32;                 // groups of 32 eigenvalues (columns)
  constexpr int WG = NW / NE;                 // warps per group in the eigenvalue-parallel phases
  extern __shared__ __align__(16) float smem[];
  float* hv = smem + L::HV;
  float* vs = smem + L::VS;
  float* work = smem + L::WORK;
  float* Em = smem + L::EM;
  float* dg = smem + L::DG;
  float* eo = smem + L::EO;
  float* e2s = smem + L::E2;
  float* betas = smem + L::BE;
  float* xpre = smem + L::XP;
  float* tpart = smem + L::TP;
  float* pvp = smem + L::PV;
  float* lamv = smem + L::LAM;
  float* theta = smem + L::TH;
  float* rho2 = smem + L::RH;
  float* sgn = smem + L::SG;
  int* ktv = reinterpret_cast<int*>(smem + L::KT);
  float* part = smem + L::PART;
  __shared__ float s_gmax, s_lo, s_hi, s_emax, s_trT;
  __shared__ double s_trace;
  __shared__ int s_flags[4];
  __shared__ int s_why;

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();          // everything below reads what the Gram kernel wrote

  // ---- 1. G = sum of the slices' partial Grams, in a fixed order -----------------------------
  float* Gs = work;    // [D][LD] staging copy
  // the summed matrix in global memory: a user's only partial as it is, else written below
  const float* gout = parts == 1 ? gpart + (size_t)b * D * D : gsum + (size_t)b * D * D;
  {
    const float4* gp = reinterpret_cast<const float4*>(gpart + (size_t)b * parts * D * D);
    int lost = 0;
    for (int s = tid; s < splits; s += NT) lost |= (gram_status[b * splits + s] != kGramStatusOk);
    int bad = 0;
    // fp32 sums in slice order.  A thread owns EPT 16-byte elements; the loads of SC slices for all
    // of them are issued before the first add: the phase is bound by their latency.
    constexpr int EPT = D * D / 4 / NT;
    constexpr int SC = (EPT >= 16) ? 2 : (EPT >= 8) ? 3 : 8;
    static_assert(EPT * NT * 4 == D * D, "whole elements");
    float4 acc[EPT];
#pragma unroll
    for (int u = 0; u < EPT; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < parts; s0 += SC) {
      float4 v[SC][EPT];
#pragma unroll
      for (int c = 0; c < SC; ++c)
#pragma unroll
        for (int u = 0; u < EPT; ++u)
          v[c][u] = (s0 + c < parts) ? __ldg(gp + (size_t)(s0 + c) * (D * D / 4) + tid + u * NT)
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int c = 0; c < SC; ++c)
#pragma unroll
        for (int u = 0; u < EPT; ++u) {
          acc[u].x += v[c][u].x; acc[u].y += v[c][u].y; acc[u].z += v[c][u].z; acc[u].w += v[c][u].w;
        }
    }
#pragma unroll
    for (int u = 0; u < EPT; ++u) {
      const int eh = tid + u * NT;
      bad |= !(isfinite(acc[u].x) && isfinite(acc[u].y) && isfinite(acc[u].z) && isfinite(acc[u].w));
      *reinterpret_cast<float4*>(Gs + (eh / (D / 4)) * LD + (eh % (D / 4)) * 4) = acc[u];
      if (parts > 1) reinterpret_cast<float4*>(gsum + (size_t)b * D * D)[eh] = acc[u];   // the residual check and the fallback read it back
    }
    if (tid < 4) s_flags[tid] = 0;
    if (tid == 0) s_why = 0;
    lost = __syncthreads_or(lost);
    bad = __syncthreads_or(bad);
    if (bad || lost) {
      const float qnan = __int_as_float(0x7fc00000);
      for (int e = tid; e < D * r; e += NT) V[(size_t)b * D * r + e] = qnan;
      for (int e = tid; e < r; e += NT) S[(size_t)b * r + e] = qnan;
      if (tid == 0 && info) info[b] = lost ? SOLAR_INFO_DEVICE_WAIT : SOLAR_INFO_NONFINITE;
      if (tid == 0 && route_taken) route_taken[b] = 0;
      return false;
    }
  }
  if (tid < 32) {
    float m = 0.f;
    double tr = 0.0;
    for (int i = tid; i < D; i += 32) {
      const float g = Gs[i * LD + i];
      m = fmaxf(m, fabsf(g));
      tr += (double)g;
    }
    m = warp_max(m);
#pragma unroll
    for (int o = 16; o; o >>= 1) tr += __shfl_xor_sync(kFull, tr, o);
    if (tid == 0) { s_gmax = m; s_trace = tr; }
  }
  __syncthreads();
  const float gmax = s_gmax;
  // Power-of-two scale that brings the largest diagonal entry into [1, 2): everything below works
  // on sc * G (exact), and the eigenvalues are divided by sc at the end.
  const float sc = gmax > 0.f ? exp2f(-(float)max(-100, min(100, ilogbf(gmax)))) : 1.f;

  bool ok = true;
  int passes = 0;
  if (route != kRouteFull && gmax > 0.f) {
    // ---- 2. Householder tridiagonalisation, the matrix in registers ---------------------------
    int k_stop = -1;                     // step at which the reduction stopped early (uniform), or -1
    {
      float a[RPT][CPT], xr[RPT], xc[CPT];
#pragma unroll
      for (int q = 0; q < RPT; ++q) {
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          const float4 t = *reinterpret_cast<const float4*>(Gs + (lane + 32 * q) * LD + 4 * (warp + NW * g));
          a[q][4 * g] = t.x * sc; a[q][4 * g + 1] = t.y * sc; a[q][4 * g + 2] = t.z * sc; a[q][4 * g + 3] = t.w * sc;
        }
        xr[q] = Gs[(lane + 32 * q) * LD] * sc;                      // column 0 at my rows ...
      }
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        const float4 t = *reinterpret_cast<const float4*>(Gs + 4 * (warp + NW * g));   // ... and (row 0) at my columns
        xc[4 * g] = t.x * sc; xc[4 * g + 1] = t.y * sc; xc[4 * g + 2] = t.z * sc; xc[4 * g + 3] = t.w * sc;
      }
      for (int e = tid; e < D * D / 4; e += NT) reinterpret_cast<float4*>(hv)[e] = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int e = tid; e < 2 * D; e += NT) xpre[e] = 0.f;
      __syncthreads();
      const float trs = (float)((double)sc * s_trace);
      float tr_rest = trs, tr_comp = 0.f;
      const float stop_tr = trs * tol.stop_trace, stop_x2 = (trs * tol.stop_couple) * (trs * tol.stop_couple);
      tri_stage<D, 0>(a, xr, xc, hv, xpre, tpart, pvp, dg, eo, betas, tid, tr_rest, tr_comp, stop_tr, stop_x2, r, k_stop);
      tri_stage<D, 1>(a, xr, xc, hv, xpre, tpart, pvp, dg, eo, betas, tid, tr_rest, tr_comp, stop_tr, stop_x2, r, k_stop);
      if constexpr (NG > 2) {
        tri_stage<D, 2>(a, xr, xc, hv, xpre, tpart, pvp, dg, eo, betas, tid, tr_rest, tr_comp, stop_tr, stop_x2, r, k_stop);
        tri_stage<D, 3>(a, xr, xc, hv, xpre, tpart, pvp, dg, eo, betas, tid, tr_rest, tr_comp, stop_tr, stop_x2, r, k_stop);
      }
      if (k_stop < 0) {
        // the last 2 x 2 block: xr holds column D-2
        if (warp == 0) {
#pragma unroll
          for (int q = 0; q < RPT; ++q) {
            if (lane + 32 * q == D - 2) dg[D - 2] = xr[q];
            if (lane + 32 * q == D - 1) eo[D - 2] = xr[q];
          }
          if (lane == 0) { eo[D - 1] = 0.f; betas[D - 2] = 0.f; betas[D - 1] = 0.f; }
        }
        if (warp == NW - 1 && lane == 31) dg[D - 1] = a[RPT - 1][CPT - 1];
      }
    }
    // T has `de` rows (all D unless the reduction stopped early), padded with zero rows to a multiple of 4
    const int de = k_stop >= 0 ? k_stop + 1 : D, de4 = (de + 3) & ~3;
    const int kb = k_stop >= 0 ? k_stop : D - 2;            // reflectors 0 .. kb-1 exist
    if (tid < de4 - de) { dg[de + tid] = 0.f; eo[de + tid] = 0.f; }
    __syncthreads();

    // ---- 3. Gershgorin interval, floored squares, trace; multisection --------------------------
    if (warp == 0) {
      float lo = 3.0e38f, hi = -3.0e38f, tr = 0.f;
      for (int i = lane; i < de; i += 32) {
        const float rad = fabsf(eo[i]) + (i > 0 ? fabsf(eo[i - 1]) : 0.f);   // eo[de-1] = 0
        lo = fminf(lo, dg[i] - rad); hi = fmaxf(hi, dg[i] + rad);
        tr += dg[i];
      }
      lo = -warp_max(-lo); hi = warp_max(hi); tr = warp_sum(tr);
      const float tn = fmaxf(fabsf(lo), fabsf(hi));
      const float fl = (tn * 1.4901161e-08f) * (tn * 1.4901161e-08f);         // (2^-26 |T|)^2
      for (int i = lane; i < de4; i += 32) e2s[i] = i > 0 ? fmaxf(eo[i - 1] * eo[i - 1], fl) : 0.f;
      if (lane == 0) {
        const float span = hi - lo;
        s_lo = lo - 1e-6f * span - 1e-30f; s_hi = hi + 1e-6f * span + 1e-30f; s_trT = tr;
      }
    }
    __syncthreads();
    const float tnorm = fmaxf(fabsf(s_lo), fabsf(s_hi));
    // Eigenvalue j = 32 * gi + lane belongs to the group gi of WG warps; every warp of the group
    // keeps the same bracket and evaluates its own interior point(s) in each step.
    const int gi = warp / WG, wg = warp % WG;
    const int j = gi * 32 + lane, jj = j < r ? j : r - 1;       // surplus lanes shadow column r-1
    float lam;
    {
      constexpr int CH = (WG >= 4) ? 1 : 2;                      // points per warp and step
      constexpr int P = CH * WG;                                 // 4 or 8 points: 5 or 9 sub-intervals
      constexpr int STEPS = (P >= 8) ? 9 : 12;                   // (P + 1)^STEPS >= 2^27
      static_assert(2 * NE * P * 32 <= RP * RP, "flags fit in the E region");
      unsigned char* flag = reinterpret_cast<unsigned char*>(Em);   // [2][NE][P][32]: count(point) > target
      const int target = de4 - 1 - jj;    // lambda_(jj-th largest) >= x  <=>  #(eigenvalues < x) <= target
      float lo = s_lo, hi = s_hi;
#pragma unroll 1
      for (int step = 0; step < STEPS; ++step) {
        const float w = (hi - lo) * (1.f / (P + 1));
        float x[CH];
        int cnt[CH];
#pragma unroll
        for (int h = 0; h < CH; ++h) x[h] = fmaf((float)(wg * CH + h + 1), w, lo);
        sturm<D, CH>(dg, e2s, x, cnt, de4 >> 2);
        unsigned char* fl = flag + (((step & 1) * NE + gi) * P) * 32;
#pragma unroll
        for (int h = 0; h < CH; ++h) fl[(wg * CH + h) * 32 + lane] = cnt[h] > target;
        __syncthreads();
        int idx = P;                       // first point above the eigenvalue
#pragma unroll
        for (int pnt = P - 1; pnt >= 0; --pnt) idx = fl[pnt * 32 + lane] ? pnt : idx;
        const float nlo = idx == 0 ? lo : fmaf((float)idx, w, lo);
        const float nhi = idx == P ? hi : fmaf((float)(idx + 1), w, lo);
        lo = nlo; hi = nhi;
      }
      lam = 0.5f * (lo + hi);
      if (wg == 0) lamv[j] = lam;
    }
    // A reduction to tridiagonal form is backward stable in the norm of G only: it fixes a kept
    // vector to an angle of a few eps |T| / gap, whatever the size of its eigenvalue.  Where a
    // gap among the kept eigenvalues is too small for the angle the storage type needs (a
    // strongly graded spectrum such as sigma_i = i^-1.5 over 128 directions), the Jacobi solve,
    // which works to an accuracy relative to each eigenvalue, takes over at once.
    __syncthreads();
    {
      int tight = 0;
      if (wg == 0 && j < r - 1) tight = (lamv[j] - lamv[j + 1]) < tol.gap_min * lamv[0];
      if (__syncthreads_or(tight)) {
        ok = false;
        if (tid == 0) s_why |= kWhyGap;
      }
    }
    float* Vc = vs;        // current vectors
    float* Vn = work;      // next (over the twisted-factorisation buffers once they are free)
    if (ok || route == kRouteTridiag) {
    // ---- 4. twisted factorisation ---------------------------------------------------------------
    // The pivots of the two triangular factorisations of T - lambda I are ratios of consecutive
    // minors: q+_i = p_{i+1} / p_i with the leading minors p of the Sturm recurrence, and
    // q-_i = t_i / t_{i+1} with the trailing minors t.  Taking them from the (rescaled) minor
    // recurrences keeps the divisions off the dependency chain, which is one FMA per step.  The
    // forward and the backward sequence run on two warps of the group; then every warp takes a
    // range of i for gamma_i and the multipliers; then two warps run the two halves of z.
    float* tf = work;                 // [D][RP] forward pivots, then the upward multipliers / values
    float* tb = work + D * RP;        // [D][RP] backward pivots, then the downward multipliers / values
    const float pfl = tnorm * 9.3132257e-10f;                                // pivot floor 2^-30 |T|
    constexpr int WB = (WG > 1) ? 1 : 0;                                     // the warp of the backward sequences
    {
      if (wg == 0) {
        float pf = 1.f, pfo = 0.f;                              // p_i, p_{i-1}
#pragma unroll 8
        for (int t = 0; t < de; ++t) {
          const float nf = fmaf(dg[t] - lam, pf, -(e2s[t] * pfo));
          float qf = __fdividef(nf, pf);
          qf = (fabsf(qf) >= pfl) ? qf : -pfl;                   // also catches NaN
          tf[t * RP + j] = qf;
          pfo = pf; pf = nf;
          if ((t & 3) == 3) {
            const unsigned mf = __float_as_uint(fmaxf(fabsf(pf), fabsf(pfo))) >> 23;
            const float sf = __uint_as_float((254u - mf) << 23);
            pf *= sf; pfo *= sf;
          }
        }
      }
      if (wg == WB) {
        float pb = 1.f, pbo = 0.f;                              // t_{i+1}, t_{i+2}
#pragma unroll 8
        for (int t = 0; t < de; ++t) {
          const int ib = de - 1 - t;
          const float nb = fmaf(dg[ib] - lam, pb, -((t > 0 ? e2s[ib + 1] : 0.f) * pbo));
          float qb = __fdividef(nb, pb);
          qb = (fabsf(qb) >= pfl) ? qb : -pfl;
          tb[ib * RP + j] = qb;
          pbo = pb; pb = nb;
          if ((t & 3) == 3) {
            const unsigned mb = __float_as_uint(fmaxf(fabsf(pb), fabsf(pbo))) >> 23;
            const float sb = __uint_as_float((254u - mb) << 23);
            pb *= sb; pbo *= sb;
          }
        }
      }
    }
    __syncthreads();
    {
      // gamma_i = q+_i + q-_i - (d_i - lambda) over my range of i; the multipliers
      // z_i = -(e_i / q+_i) z_{i+1} going up, z_i = -(e_{i-1} / q-_i) z_{i-1} going down
      const int IR = (de + WG - 1) / WG, i1 = min((wg + 1) * IR, de);
      float best = 3.0e38f;
      int kbest = 0;
#pragma unroll 8
      for (int i = wg * IR; i < i1; ++i) {
        const float qf = tf[i * RP + j], qb = tb[i * RP + j];
        const float gam = fabsf((qf + qb) - (dg[i] - lam));
        if (gam < best) { best = gam; kbest = i; }
        tf[i * RP + j] = -__fdividef(eo[i], qf);
        tb[i * RP + j] = i > 0 ? -__fdividef(eo[i - 1], qb) : 0.f;
      }
      part[wg * RP + j] = best;
      reinterpret_cast<int*>(part)[(NW + wg) * RP + j] = kbest;
    }
    __syncthreads();
    int kt = 0;
    {
      float best = 3.0e38f;
#pragma unroll
      for (int w2 = 0; w2 < WG; ++w2) {
        const float bv = part[w2 * RP + j];
        const int bk = reinterpret_cast<const int*>(part)[(NW + w2) * RP + j];
        if (bv < best) { best = bv; kt = bk; }                   // ranges ascend: the lowest i wins a tie
      }
    }
    __syncthreads();
    {
      // z_kt = 1; the values above the twist overwrite tf, those below it tb (no branches: a lane
      // that has not reached its twist index yet keeps z = 1)
      if (wg == 0) {
        float zu = 1.f, ss = 0.f;
#pragma unroll 8
        for (int iu = de - 2; iu >= 0; --iu) {
          const float mu = tf[iu * RP + j];
          zu = (iu < kt) ? zu * mu : 1.f;
          ss = fmaf(zu, (iu < kt) ? zu : 0.f, ss);
          tf[iu * RP + j] = zu;
        }
        part[j] = ss;
        ktv[j] = kt;
      }
      if (wg == WB) {
        float zd = 1.f, ss = 0.f;
#pragma unroll 8
        for (int t = 1; t < de; ++t) {
          const float md = tb[t * RP + j];
          zd = (t > kt) ? zd * md : 1.f;
          ss = fmaf(zd, (t > kt) ? zd : 0.f, ss);
          tb[t * RP + j] = zd;
        }
        part[RP + j] = ss;
      }
    }
    __syncthreads();
    if (wg == 0) sgn[j] = rsqrtf(1.f + part[j] + part[RP + j]);   // 1 / |z|
    __syncthreads();

    // ---- 5. back-transformation: v = H_0 H_1 ... H_{D-3} z ------------------------------------
    // Four threads per vector, each with a quarter of the rows in registers; the reflector's
    // inner product is completed by two shuffles.  Reflector k is zero at rows <= k, so the
    // quarters need no conditions.
    {
      constexpr int RB = D / 4;                   // rows per thread
      constexpr int VPP = NT / 4;                 // vectors per pass
      constexpr int NPASS = (RP + VPP - 1) / VPP;
      static_assert(NPASS * VPP >= RP, "every vector is transformed");
#pragma unroll 1
      for (int pass = 0; pass < NPASS; ++pass) {
        const int jv = pass * VPP + (tid >> 2), qt = tid & 3;
        const bool act = jv < RP;
        const int jc = act ? jv : 0;
        const int ktj = ktv[jc];
        const float zn = sgn[jc];
        float z[RB];
#pragma unroll
        for (int u = 0; u < RB; ++u) {
          const int i = qt * RB + u;
          const float upv = tf[i * RP + jc], dnv = tb[i * RP + jc];
          z[u] = i < de ? (i < ktj ? upv : i > ktj ? dnv : 1.f) * zn : 0.f;
        }
#pragma unroll 2
        for (int k = kb - 1; k >= 0; --k) {
          const float beta = betas[k];
          const float4* h4 = reinterpret_cast<const float4*>(hv + k * D + qt * RB);
          float4 h[RB / 4];
          float d0 = 0.f, d1 = 0.f;
#pragma unroll
          for (int u = 0; u < RB / 4; ++u) {
            h[u] = h4[u];
            d0 = fmaf(h[u].x, z[4 * u], d0);     d1 = fmaf(h[u].y, z[4 * u + 1], d1);
            d0 = fmaf(h[u].z, z[4 * u + 2], d0); d1 = fmaf(h[u].w, z[4 * u + 3], d1);
          }
          float dt = d0 + d1;
          dt += __shfl_xor_sync(kFull, dt, 1);
          dt += __shfl_xor_sync(kFull, dt, 2);
          const float c = -beta * dt;
#pragma unroll
          for (int u = 0; u < RB / 4; ++u) {
            z[4 * u] = fmaf(c, h[u].x, z[4 * u]);         z[4 * u + 1] = fmaf(c, h[u].y, z[4 * u + 1]);
            z[4 * u + 2] = fmaf(c, h[u].z, z[4 * u + 2]); z[4 * u + 3] = fmaf(c, h[u].w, z[4 * u + 3]);
          }
        }
        if (act) {
#pragma unroll
          for (int u = 0; u < RB; ++u) vs[(qt * RB + u) * RP + jv] = z[u];
        }
      }
    }
    __syncthreads();
    // The long serial part is over: the next kernel may start launching -- unless the process runs
    // many requests at once, where its parked CTAs are better kept out a little longer (after the
    // certificate: 7.65 -> 7.59 us per step in flight, at 0.4 us of a single call's latency).
    if (!late_trigger) pdl_trigger();

    // G back into shared memory (over the reflectors), for the residuals
    float* Gsm = hv;   // [D][D], sc * G
    for (int e = tid; e < D * D / 4; e += NT) {
      float4 g = reinterpret_cast<const float4*>(gout)[e];
      g.x *= sc; g.y *= sc; g.z *= sc; g.w *= sc;
      reinterpret_cast<float4*>(Gsm)[e] = g;
    }

    // ---- 6. orthogonalisation passes while V^T V - I is above the rounding level ---------------
    // Column-parallel: lane = column(s) c, c + 32; a warp takes RP / NW rows a of E.
    constexpr int AW = RP / NW;
    for (;;) {
      float acc[NE][AW];
#pragma unroll
      for (int h = 0; h < NE; ++h)
#pragma unroll
        for (int u = 0; u < AW; ++u) acc[h][u] = 0.f;
      const int a0 = warp * AW;
#pragma unroll 8
      for (int i = 0; i < D; ++i) {
        float av[AW];
        if (AW >= 4) {
#pragma unroll
          for (int u = 0; u < AW; u += 4) {
            const float4 t = *reinterpret_cast<const float4*>(Vc + i * RP + a0 + u);
            av[u] = t.x; av[u + 1] = t.y; av[u + 2] = t.z; av[u + 3] = t.w;
          }
        } else {
#pragma unroll
          for (int u = 0; u < AW; ++u) av[u] = Vc[i * RP + a0 + u];
        }
#pragma unroll
        for (int h = 0; h < NE; ++h) {
          const float vc = Vc[i * RP + 32 * h + lane];
#pragma unroll
          for (int u = 0; u < AW; ++u) acc[h][u] = fmaf(av[u], vc, acc[h][u]);
        }
      }
      float emax = 0.f;
#pragma unroll
      for (int h = 0; h < NE; ++h)
#pragma unroll
        for (int u = 0; u < AW; ++u) {
          const int a = a0 + u, c = 32 * h + lane;
          float e = acc[h][u] - (a == c ? 1.f : 0.f);
          if (a >= r || c >= r) e = 0.f;               // surplus columns are copies of column r-1
          Em[a * RP + c] = e;
          emax = fmaxf(emax, fabsf(e));
        }
      emax = warp_max(emax);
      if (lane == 0) part[warp] = emax;
      __syncthreads();
      if (tid == 0) {
        float m = 0.f;
        for (int w = 0; w < NW; ++w) m = fmaxf(m, part[w]);
        s_emax = m;
      }
      __syncthreads();
      const float em = s_emax;
      if (em <= tol.ortho) break;                       // orthonormal to rounding
      if (passes == 6 || !(em <= 0.98f)) { ok = false; if (tid == 0) s_why |= kWhyOrtho; break; }
      ++passes;
      // One pass of Gram-Schmidt against the ORIGINAL earlier columns (larger eigenvalues, the
      // better determined vectors): v_c <- (v_c - sum_{a<c} E_ac v_a) / |.|.  A later column never
      // changes an earlier one, so a poorly separated pair cannot damage its neighbours; for
      // two vectors the pass is exact, for more it converges quadratically like the symmetric
      // form.  Rows i of V' for this warp: D / NW of them; lane = column(s).
      float ecol[NE][RP], scol[NE];
#pragma unroll
      for (int h = 0; h < NE; ++h) {
        const int c = 32 * h + lane;
        float nn = 1.f;
#pragma unroll
        for (int a = 0; a < RP; ++a) {
          const float e = Em[a * RP + c];
          ecol[h][a] = a < c ? e : 0.f;
          nn += a < c ? -e * e : (a == c ? e : 0.f);
        }
        scol[h] = rsqrtf(fmaxf(nn, 1e-6f));
      }
      for (int i = warp; i < D; i += NW) {
        float o[NE];
#pragma unroll
        for (int h = 0; h < NE; ++h) o[h] = 0.f;
#pragma unroll
        for (int a = 0; a < RP; a += 4) {
          const float4 t = *reinterpret_cast<const float4*>(Vc + i * RP + a);
#pragma unroll
          for (int h = 0; h < NE; ++h) {
            o[h] = fmaf(t.x, ecol[h][a], o[h]);     o[h] = fmaf(t.y, ecol[h][a + 1], o[h]);
            o[h] = fmaf(t.z, ecol[h][a + 2], o[h]); o[h] = fmaf(t.w, ecol[h][a + 3], o[h]);
          }
        }
#pragma unroll
        for (int h = 0; h < NE; ++h)
          Vn[i * RP + 32 * h + lane] = (Vc[i * RP + 32 * h + lane] - o[h]) * scol[h];
      }
      __syncthreads();
      float* t = Vc; Vc = Vn; Vn = t;
      // With E = L + diag + L^T the pass leaves (I - L)(I + E)(I - L^T) = I + diag - L L^T - L^2 -
      // (L^T)^2 + O(E^3), and the scaling removes the diagonal: what remains off the diagonal is
      // below 3 r max|E|^2.  Where that is a quarter of the bound, V^T V is not formed again.
      if (3.f * (float)r * em * em <= 0.25f * tol.ortho) break;
    }
    __syncthreads();      // G is staged; E and the vectors are settled

    // ---- 7. Rayleigh quotients and residuals against G; certification ------------------------
    if (ok || route == kRouteTridiag) {
      constexpr int RW = D / NW;        // rows of Y = G V per warp
      float y[NE][RW];
#pragma unroll
      for (int h = 0; h < NE; ++h)
#pragma unroll
        for (int u = 0; u < RW; ++u) y[h][u] = 0.f;
      const int i0 = warp * RW;
#pragma unroll 2
      for (int k = 0; k < D; k += 4) {
        float vk[NE][4];
#pragma unroll
        for (int h = 0; h < NE; ++h)
#pragma unroll
          for (int u = 0; u < 4; ++u) vk[h][u] = Vc[(k + u) * RP + 32 * h + lane];
#pragma unroll
        for (int u = 0; u < RW; ++u) {
          const float4 g = *reinterpret_cast<const float4*>(Gsm + (i0 + u) * D + k);
#pragma unroll
          for (int h = 0; h < NE; ++h) {
            y[h][u] = fmaf(g.x, vk[h][0], y[h][u]); y[h][u] = fmaf(g.y, vk[h][1], y[h][u]);
            y[h][u] = fmaf(g.z, vk[h][2], y[h][u]); y[h][u] = fmaf(g.w, vk[h][3], y[h][u]);
          }
        }
      }
      float vown[NE][RW];
#pragma unroll
      for (int h = 0; h < NE; ++h) {
        float t = 0.f;
#pragma unroll
        for (int u = 0; u < RW; ++u) {
          vown[h][u] = Vc[(i0 + u) * RP + 32 * h + lane];
          t = fmaf(vown[h][u], y[h][u], t);
        }
        part[warp * RP + 32 * h + lane] = t;
      }
      __syncthreads();
      if (tid < RP) {
        float t = 0.f;
        for (int w = 0; w < NW; ++w) t += part[w * RP + tid];
        theta[tid] = t;
      }
      __syncthreads();
#pragma unroll
      for (int h = 0; h < NE; ++h) {
        const float th = theta[32 * h + lane];
        float t = 0.f;
#pragma unroll
        for (int u = 0; u < RW; ++u) {
          const float d = fmaf(-th, vown[h][u], y[h][u]);
          t = fmaf(d, d, t);
        }
        part[warp * RP + 32 * h + lane] = t;
      }
      __syncthreads();
      if (tid < RP) {
        float t = 0.f;
        for (int w = 0; w < NW; ++w) t += part[w * RP + tid];
        rho2[tid] = t;
      }
      __syncthreads();
      int good = 1;
      if (tid < r) {
        const float th1 = theta[0], thi = theta[tid];
        float gap = 3.0e38f;
        if (tid > 0) gap = fminf(gap, theta[tid - 1] - thi);
        if (tid < r - 1) gap = fminf(gap, thi - theta[tid + 1]);
        const float resn = sqrtf(rho2[tid]);
        const bool res_ok = resn <= fmaxf(tol.eps_vec * gap, tol.floor_rel * th1);
        // T is similar to sc * G: the traces agree to rounding
        const float trG = (float)((double)sc * s_trace);
        const bool tr_ok = fabsf(s_trT - trG) <= 1e-4f * fabsf(trG) && isfinite(thi) && isfinite(resn);
        if (!res_ok) atomicOr(&s_why, kWhyResidual);
        if (!tr_ok) atomicOr(&s_why, kWhyTrace);
        good = res_ok && tr_ok;
      }
      ok = __syncthreads_and(good) && ok;
    }

    }   // the gaps allow the tridiagonal route

    if (ok || route == kRouteTridiag) {
      if (late_trigger) pdl_trigger();
      // singular values (non-increasing: a Rayleigh quotient may pass its neighbour by a rounding
      // error), sign gauge, output
      if (tid < RP) {
        const int j = tid < r ? tid : r - 1;
        float m = theta[j];
        for (int q = 0; q < j; ++q) m = fminf(m, theta[q]);
        float best = -1.f, lead = 1.f;
        for (int i = 0; i < D; ++i) {
          const float v = Vc[i * RP + j];
          if (fabsf(v) > best) { best = fabsf(v); lead = v; }   // strict: lowest index wins a tie
        }
        sgn[tid] = lead < 0.f ? -1.f : 1.f;
        const float sv = sqrtf(fmaxf(m, 0.f) / sc);
        rho2[tid] = sv;
        if (tid < r) S[(size_t)b * r + tid] = sv;
      }
      __syncthreads();
      for (int e = tid; e < D * r; e += NT) {
        const int i = e / r, j = e % r;
        V[(size_t)b * D * r + e] = Vc[i * RP + j] * sgn[j];
      }
      if (want_vs) {
        const int rp = (r + 3) & ~3;
        float* vsig = smem;                            // over G: the residuals are done
        for (int e = tid; e < D * rp; e += NT) {
          const int i = e / rp, j = e % rp;
          vsig[e] = j < r ? (Vc[i * RP + j] * sgn[j]) * rho2[j] : 0.f;
        }
      }
      if (tid == 0) {
        if (info) info[b] = ok ? 0 : SOLAR_INFO_NOT_CERTIFIED;
        if (route_taken) route_taken[b] = kRouteTridiag | (passes << 16) | (s_why << 24);
      }
      return want_vs;
    }
    __syncthreads();
  }

  // ---- fallback (or the caller's choice): Jacobi on the whole matrix ---------------------------
  for (int e = tid; e < D * D / 4; e += NT) {
    float4 g = reinterpret_cast<const float4*>(gout)[e];
    g.x *= sc; g.y *= sc; g.z *= sc; g.w *= sc;
    *reinterpret_cast<float4*>(smem + (e / (D / 4)) * LD + (e % (D / 4)) * 4) = g;
  }
  __syncthreads();
  const float thr_abs2 = (kTolAbs * gmax * sc) * (kTolAbs * gmax * sc);
  full_jacobi_route<D, NT>(smem, s_flags, b, tid, r, sc, thr_abs2, tol.sweep_stop * tol.sweep_stop, s_why,
                           sweep_cap, S, V, info, route_taken);
  return false;
}

// ---- optional epilogue: the factor-token projections of Eq. 11 for this user ---------------
// Key_r = (V Sigma)^T W_K, Value_r = (V Sigma)^T W_V and the folded score operand
// T = scale * W_Q Key_r^T, written to the attention workspace in the layout and with the
// summation order of the stand-alone projection kernel, so that a forward pass which ends its
// eigensolver CTAs with this epilogue needs one launch less and gives the same bits.
struct FuseArgs {
  const void* Wq; const void* Wk; const void* Wv;
  float scale;
  char* ws;            // attention workspace (all users)
  AttnWs lay;
  int mode;            // 0: no epilogue; 1: weights are bf16; 2: weights are fp32
  int write_f32;       // also write the fp32 copies T and Value_r (read by the FFMA attention kernel)
  int late_trigger;    // release the next kernel after the certificate instead of before the residuals
};

// Stages W[D][D] (bf16 or fp32 in global memory) as fp32 in shared memory, as it is or
// transposed.  All loads of a thread are issued before the first store.
template <int D, int NT, bool TRANSPOSE>
__device__ __forceinline__ void stage_weight_any(const void* __restrict__ W, int mode, float* __restrict__ Ws,
                                                 int tid) {
  constexpr int NV = D * D / 8 / NT;              // 8-element pieces per thread
  static_assert(NV * NT * 8 == D * D, "whole pieces");
  float x[NV][8];
  if (mode == 1) {
    const uint4* w = static_cast<const uint4*>(W);
    uint4 raw[NV];
#pragma unroll
    for (int n = 0; n < NV; ++n) raw[n] = __ldg(w + tid + n * NT);
#pragma unroll
    for (int n = 0; n < NV; ++n) {
      const uint32_t u[4] = {raw[n].x, raw[n].y, raw[n].z, raw[n].w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        x[n][2 * q] = __uint_as_float(u[q] << 16);
        x[n][2 * q + 1] = __uint_as_float(u[q] & 0xffff0000u);
      }
    }
  } else {
    const float4* w = static_cast<const float4*>(W);
#pragma unroll
    for (int n = 0; n < NV; ++n) {
      const float4 lo = __ldg(w + 2 * (tid + n * NT)), hi = __ldg(w + 2 * (tid + n * NT) + 1);
      x[n][0] = lo.x; x[n][1] = lo.y; x[n][2] = lo.z; x[n][3] = lo.w;
      x[n][4] = hi.x; x[n][5] = hi.y; x[n][6] = hi.z; x[n][7] = hi.w;
    }
  }
#pragma unroll
  for (int n = 0; n < NV; ++n) {
    const int e0 = (tid + n * NT) * 8;            // element e0 = row * D + col
    if (!TRANSPOSE) {
      *reinterpret_cast<float4*>(Ws + e0) = make_float4(x[n][0], x[n][1], x[n][2], x[n][3]);
      *reinterpret_cast<float4*>(Ws + e0 + 4) = make_float4(x[n][4], x[n][5], x[n][6], x[n][7]);
    } else {
      const int row = e0 / D, col = e0 % D;
#pragma unroll
      for (int u = 0; u < 8; ++u) Ws[(col + u) * D + row] = x[n][u];
    }
  }
}

// 16-byte pieces of a packed bf16 operand row: eight fp32 values as their high halves (h = 0)
// or as what the high halves leave over (h = 1).
__device__ __forceinline__ uint4 pack8_bf16(const float (&x)[8], int h) {
  uint32_t w[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    float a = x[2 * q], c = x[2 * q + 1];
    if (h) {
      a -= __bfloat162float(__float2bfloat16_rn(a));
      c -= __bfloat162float(__float2bfloat16_rn(c));
    }
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, c);
    w[q] = *reinterpret_cast<const uint32_t*>(&v);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// vs_ready: V Sigma of this user already lies at sm[0 .. D * rp) (pitch rp = r rounded up to 4,
// zero in the padding), left there by the eigensolver; otherwise it is read back from S and V.
template <int D, int NT>
__device__ __forceinline__ void prepare_epilogue(float* __restrict__ sm, int b, int r, const float* __restrict__ S,
                                                 const float* __restrict__ V, const FuseArgs& fa, bool vs_ready,
                                                 int tid) {
  const int rp = (r + 3) & ~3;          // token pitch: rows of VS / KrT are read 4 at a time
  float* VS = sm;                       // [D][rp]  V Sigma (zero in the padding)
  float* KrT = VS + D * rp;             // [D][rp]  Key_r^T; later Value_r^T
  float* W0 = KrT + D * rp;             // [D][D]   W_K, then W_V
  float* W1 = W0 + D * D;               // [D][D]   W_Q^T; later T^T [r][D]
  char* wsb = fa.ws + (size_t)b * fa.lay.per_user;
  float* Tf = reinterpret_cast<float*>(wsb + fa.lay.tf_off);
  float* Vr = reinterpret_cast<float*>(wsb + fa.lay.vr_off);
  __nv_bfloat16* Tpk = reinterpret_cast<__nv_bfloat16*>(wsb + fa.lay.tpk_off);
  __nv_bfloat16* Vpk = reinterpret_cast<__nv_bfloat16*>(wsb + fa.lay.vpk_off);
  const int nt4 = rp / 4;               // groups of four tokens
  const int ntile = nt4 * (D / 4);      // 4 x 4 output tiles of each of the three products
  constexpr int MAXT = 2;               // tiles per thread (kept in registers across a barrier)
  const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);

  if (D >= 64 && fa.mode == 1 && !fa.write_f32) {
    // bf16 weights: the three products on the tensor cores
    if (!vs_ready) {
      for (int e = tid; e < D * rp; e += NT) {
        const int k = e / rp, i = e % rp;
        VS[e] = i < r ? __ldcg(V + ((size_t)b * D + k) * r + i) * __ldcg(S + (size_t)b * r + i) : 0.f;
      }
      __syncthreads();
    }
    pmma::project<(D >= 64 ? D : 64), NT>(reinterpret_cast<unsigned char*>(sm), r, fa.Wq, fa.Wk, fa.Wv, fa.scale, Tpk, Vpk,
                                          nullptr, nullptr, (r + 15) & ~15, tid);
    return;
  }
  stage_weight_any<D, NT, false>(fa.Wk, fa.mode, W0, tid);
  stage_weight_any<D, NT, true>(fa.Wq, fa.mode, W1, tid);
  if (!vs_ready)
    for (int e = tid; e < D * rp; e += NT) {
      const int k = e / rp, i = e % rp;
      // written earlier by this CTA: read through the L2, not the non-coherent path
      VS[e] = i < r ? __ldcg(V + ((size_t)b * D + k) * r + i) * __ldcg(S + (size_t)b * r + i) : 0.f;
    }
  // Zero padding of the packed operands, 16 bytes at a time.  The tensor-core attention kernel
  // multiplies over np = 16 ceil(r / 16) token slots only (slots r .. r8-1, r8 = r rounded up to
  // 8, are written as zeros with the data below); the FFMA kernels' callers want all 64.
  const int r8 = (r + 7) & ~7;
  const int pad_to = fa.write_f32 ? kTokenSlots : ((r + 15) & ~15);
  for (int e = tid; e < 2 * (pad_to - r8) * (D / 8); e += NT) {
    const int h = e / ((pad_to - r8) * (D / 8)), rem = e % ((pad_to - r8) * (D / 8));
    reinterpret_cast<uint4*>(Tpk + ((size_t)h * kTokenSlots + r8) * D)[rem] = z4;
  }
  for (int e = tid; e < 2 * D * ((pad_to - r8) / 8); e += NT) {
    const int row = e / ((pad_to - r8) / 8), c = e % ((pad_to - r8) / 8);
    reinterpret_cast<uint4*>(Vpk + (size_t)row * kTokenSlots + r8)[c] = z4;      // row runs over [2][D]
  }
  __syncthreads();
  // acc[a][c] = sum_k VS[k][i0 + a] W0[k][j0 + c]: a 4 x 4 tile per thread, two 16-byte reads per
  // 16 FMAs, every output summed over k in ascending order
  auto project = [&](float (&acc)[4][4], int i0, int j0) {
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[a][c] = 0.f;
#pragma unroll 4
    for (int k = 0; k < D; ++k) {
      const float4 w = *reinterpret_cast<const float4*>(W0 + k * D + j0);
      const float4 v = *reinterpret_cast<const float4*>(VS + k * rp + i0);
      const float ww[4] = {w.x, w.y, w.z, w.w}, vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] = fmaf(vv[a], ww[c], acc[a][c]);
    }
  };
  // Key_r^T [j][i]
  for (int t = tid; t < ntile; t += NT) {
    const int j0 = (t % (D / 4)) * 4, i0 = (t / (D / 4)) * 4;
    float acc[4][4];
    project(acc, i0, j0);
#pragma unroll
    for (int c = 0; c < 4; ++c)
      *reinterpret_cast<float4*>(KrT + (j0 + c) * rp + i0) = make_float4(acc[0][c], acc[1][c], acc[2][c], acc[3][c]);
  }
  __syncthreads();
  // T[k][i] = scale * sum_j Wq[k][j] Key_r[i][j]: tile of four rows k and four tokens i; kept in
  // registers until W_Q is done with, then laid down over it as T^T [i][D] (the packed rows)
  float tacc[MAXT][4][4];
#pragma unroll
  for (int n = 0; n < MAXT; ++n) {
    const int t = tid + n * NT;
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int c = 0; c < 4; ++c) tacc[n][a][c] = 0.f;
    if (t < ntile) {
      const int i0 = (t % nt4) * 4, k0 = (t / nt4) * 4;
#pragma unroll 4
      for (int j = 0; j < D; ++j) {
        const float4 w = *reinterpret_cast<const float4*>(W1 + j * D + k0);      // W_Q[k0 ..][j]
        const float4 kr = *reinterpret_cast<const float4*>(KrT + j * rp + i0);
        const float ww[4] = {w.x, w.y, w.z, w.w}, kk[4] = {kr.x, kr.y, kr.z, kr.w};
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int c = 0; c < 4; ++c) tacc[n][a][c] = fmaf(ww[a], kk[c], tacc[n][a][c]);
      }
    }
  }
  __syncthreads();
  stage_weight_any<D, NT, false>(fa.Wv, fa.mode, W0, tid);       // W_K is done with
#pragma unroll
  for (int n = 0; n < MAXT; ++n) {
    const int t = tid + n * NT;
    if (t < ntile) {
      const int i0 = (t % nt4) * 4, k0 = (t / nt4) * 4;
#pragma unroll
      for (int c = 0; c < 4; ++c)
        *reinterpret_cast<float4*>(W1 + (i0 + c) * D + k0) =
            make_float4(tacc[n][0][c] * fa.scale, tacc[n][1][c] * fa.scale, tacc[n][2][c] * fa.scale,
                        tacc[n][3][c] * fa.scale);
    }
  }
  __syncthreads();
  // T^T out: 16-byte pieces of the packed rows (tokens r .. r8-1 are zero rows), and the fp32 copy
  for (int e = tid; e < 2 * r8 * (D / 8); e += NT) {
    const int h = e / (r8 * (D / 8)), rem = e % (r8 * (D / 8)), i = rem / (D / 8), c = rem % (D / 8);
    const float4 lo = *reinterpret_cast<const float4*>(W1 + i * D + 8 * c);
    const float4 hi = *reinterpret_cast<const float4*>(W1 + i * D + 8 * c + 4);
    float x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    if (i >= r) {
#pragma unroll
      for (int u = 0; u < 8; ++u) x[u] = 0.f;
    }
    reinterpret_cast<uint4*>(Tpk + ((size_t)h * kTokenSlots + i) * D)[c] = pack8_bf16(x, h);
  }
  if (fa.write_f32)
    for (int e = tid; e < D * r; e += NT) Tf[e] = W1[(e % r) * D + e / r];
  // Value_r, kept in registers until Key_r^T is done with, then laid down over it as
  // Value_r^T [j][rp] (the packed operand's rows)
#pragma unroll
  for (int n = 0; n < MAXT; ++n) {
    const int t = tid + n * NT;
    if (t < ntile) project(tacc[n], (t / (D / 4)) * 4, (t % (D / 4)) * 4);
  }
  __syncthreads();
#pragma unroll
  for (int n = 0; n < MAXT; ++n) {
    const int t = tid + n * NT;
    if (t < ntile) {
      const int j0 = (t % (D / 4)) * 4, i0 = (t / (D / 4)) * 4;
#pragma unroll
      for (int c = 0; c < 4; ++c)
        *reinterpret_cast<float4*>(KrT + (j0 + c) * rp + i0) =
            make_float4(tacc[n][0][c], tacc[n][1][c], tacc[n][2][c], tacc[n][3][c]);
    }
  }
  __syncthreads();
  for (int e = tid; e < 2 * D * (r8 / 8); e += NT) {
    const int h = e / (D * (r8 / 8)), rem = e % (D * (r8 / 8)), j = rem / (r8 / 8), c = rem % (r8 / 8);
    float x[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) x[u] = (8 * c + u < r) ? KrT[j * rp + 8 * c + u] : 0.f;
    reinterpret_cast<uint4*>(Vpk + ((size_t)h * D + j) * kTokenSlots)[c] = pack8_bf16(x, h);
  }
  if (fa.write_f32)
    for (int e = tid; e < r * D; e += NT) Vr[e] = KrT[(e % D) * rp + e / D];
}

template <int D, int RP>
__global__ void __launch_bounds__(TriCfg<D>::NT, 1)
eig_tridiag_kernel(const float* __restrict__ gpart, const int* __restrict__ gram_status, int parts, int splits,
                   float* __restrict__ gsum, int r, int route, int sweep_cap, TriTol tol,
                   float* __restrict__ S, float* __restrict__ V, int* __restrict__ info,
                   int* __restrict__ route_taken, FuseArgs fa) {
  const bool vs_ready = eig_user<D, RP>(gpart, gram_status, parts, splits, gsum, r, route, sweep_cap, tol, fa.mode != 0, fa.late_trigger != 0, S, V,
                                        info, route_taken);
  if (fa.mode != 0) {
    extern __shared__ __align__(16) float smem[];
    __syncthreads();                    // S and V of this user are written (and visible to the CTA)
    prepare_epilogue<D, TriCfg<D>::NT>(smem, blockIdx.x, r, S, V, fa, vs_ready, threadIdx.x);
  }
}

template <int D, int RP>
cudaError_t launch_tri(int B, int r, int route, int sweep_cap, TriTol tol, const float* gpart,
                       const int* gram_status, int parts, int splits, float* gsum, float* S, float* V, int* info,
                       int* route_taken, const FuseArgs& fa, cudaStream_t st) {
  using L = TriSmem<D, RP>;
  static bool limits_set[kMaxDevicesCached] = {};
  const cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&eig_tridiag_kernel<D, RP>), L::BYTES,
                                          limits_set);
  if (e != cudaSuccess) return e;
  return launch_pdl(eig_tridiag_kernel<D, RP>, dim3(B), dim3(TriCfg<D>::NT), L::BYTES, st, gpart, gram_status,
                    parts, splits, gsum, r, route, sweep_cap, tol, S, V, info, route_taken, fa);
}

}  // namespace

cudaError_t launch_eig_tridiag(int B, int d, int r, solar_dtype_t dt, int route, int sweep_cap,
                               const float* gpart, const int* gram_status, int parts, int splits, float* gsum,
                               float* S, float* V, int* info, int* route_taken, const EigFuse* fuse,
                               cudaStream_t st) {
  FuseArgs fa = {};
  if (fuse != nullptr) {
    fa.Wq = fuse->Wq; fa.Wk = fuse->Wk; fa.Wv = fuse->Wv; fa.scale = fuse->scale;
    fa.ws = fuse->attn_ws; fa.lay = attn_ws_layout(d, r);
    fa.mode = (dt == SOLAR_BF16) ? 1 : 2;
    fa.write_f32 = !attn_umma_supported(d, dt);
    fa.late_trigger = slice_limit() > 0;
  }
  TriTol tol;
  if (dt == SOLAR_BF16) {
    tol.eps_vec = 1e-3f; tol.floor_rel = 64.f * kUnit; tol.ortho = 4e-6f; tol.sweep_stop = 1e-3f;
    tol.gap_min = 4.f * kUnit / 1e-2f;      // angle 1e-2: outputs are rounded to bf16 (2^-9)
    tol.stop_trace = 1.9073486e-06f; tol.stop_couple = 2.3841858e-07f;     // 2^-19, 2^-22
  } else {
    tol.eps_vec = 1e-5f; tol.floor_rel = 32.f * kUnit; tol.ortho = 2e-6f; tol.sweep_stop = 1e-5f;
    tol.gap_min = 4.f * kUnit / 1e-3f;
    tol.stop_trace = 1.1920929e-07f; tol.stop_couple = 2.9802322e-08f;     // 2^-23, 2^-25
  }
  const bool wide = r > 32;
  switch (d) {
    case 32:
      return launch_tri<32, 32>(B, r, route, sweep_cap, tol, gpart, gram_status, parts, splits, gsum, S, V, info, route_taken, fa, st);
    case 64:
      return wide ? launch_tri<64, 64>(B, r, route, sweep_cap, tol, gpart, gram_status, parts, splits, gsum, S, V, info, route_taken, fa, st)
                  : launch_tri<64, 32>(B, r, route, sweep_cap, tol, gpart, gram_status, parts, splits, gsum, S, V, info, route_taken, fa, st);
    case 128:
      return wide ? launch_tri<128, 64>(B, r, route, sweep_cap, tol, gpart, gram_status, parts, splits, gsum, S, V, info, route_taken, fa, st)
                  : launch_tri<128, 32>(B, r, route, sweep_cap, tol, gpart, gram_status, parts, splits, gsum, S, V, info, route_taken, fa, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace solar
