// Batched symmetric eigensolver, tridiagonal route: the top-r eigenpairs of every Gram matrix
// G_b = H_b^T H_b (Eq. 9 without U: s_i = sqrt(lambda_i), V = eigenvectors) by the classical
// dense-symmetric chain, one CTA per user, sized so that a user costs a few tens of thousands
// of warp instructions instead of a few hundred thousand for a Jacobi solve:
//
//   1. G = sum of the slices' partial Grams (fixed order), scaled by a power of two.
//   2. Householder tridiagonalisation T = Q^T G Q with the matrix held in REGISTERS: one row
//      (d = 32, 128) or two rows (d = 64) per lane of the warps that take part, so the
//      symmetric matrix-vector product and the rank-2 update of a step are lane-local FMAs on
//      statically indexed registers; a step needs two reductions (the column norm and p^T v)
//      and, with one warp, no CTA barrier at all.
//   3. The r largest eigenvalues of T by multisection on Sturm counts (one lane per
//      eigenvalue, three interior points per step: two bits per step), the counts taken from
//      the three-term recurrence of the leading principal minors with a power-of-two rescale
//      every four steps -- one FMA per step on the dependency chain instead of a division.
//   4. One eigenvector per lane from the twisted factorisation of T - lambda I (forward and
//      backward pivot sequences, twist at the smallest |gamma_k|): inverse iteration from the
//      best unit vector, O(d) per vector, no pivoting.
//   5. Back-transformation V = Q Z, each lane applying the d-2 reflectors to its own vector
//      held in registers.
//   6. A first-order symmetric orthogonalisation V <- V (I - (V^T V - I)/2), repeated while
//      V^T V - I is above the rounding level (vectors of close eigenvalues come out of step 4
//      with a mutual error of order eps |T| / gap).
//   7. Rayleigh quotients theta_i = v_i^T G v_i and residuals G v_i - theta_i v_i against the
//      ORIGINAL G: the result is accepted only if every residual is small against its gap (or
//      at the rounding floor), V^T V = I to rounding, and trace(T) = trace(G); otherwise the
//      CTA runs the parallel Jacobi eigensolver on the whole matrix, which is valid for any
//      spectrum (clusters of equal eigenvalues, rank(H) < r, ...).
#include "eig_jacobi.cuh"

namespace solar {

namespace {

constexpr unsigned kFull = 0xffffffffu;

template <int D> struct TriCfg {
  static constexpr int NT = (D == 128) ? 256 : 128;   // threads of the CTA
  static constexpr int NW = NT / 32;
  static constexpr int TW = (D == 128) ? 4 : 1;       // warps that hold the matrix while it is reduced
  static constexpr int RPL = (D == 64) ? 2 : 1;       // rows per lane
  static constexpr int LD = D + 4;                    // pitch of the staged row-major G
  static constexpr int NB = D / 4;                    // 4-column blocks of a row
  static_assert(TW * 32 * RPL == D, "every row has an owner");
};

// Shared-memory layout (floats) for subspace width RP = 32 * ceil(r / 32).
template <int D, int RP> struct TriSmem {
  using C = TriCfg<D>;
  static constexpr int HV = 0;                                   // [D][D] reflector k in row k; later G
  static constexpr int VS = HV + D * D;                          // [D][RP] tridiagonal vectors, then V
  static constexpr int WORK_FLOATS = (D * C::LD > 2 * D * RP) ? D * C::LD : 2 * D * RP;
  static constexpr int WORK = VS + D * RP;                       // staged G | tf, tb [D][RP] | V'
  static constexpr int EM = WORK + WORK_FLOATS;                  // [RP][RP] V^T V - I
  static constexpr int DG = EM + RP * RP;                        // [D] diagonal of T
  static constexpr int EO = DG + D;                              // [D] off-diagonal: e[k] couples k, k+1
  static constexpr int E2 = EO + D;                              // [D] e2s[i] = e[i-1]^2 (floored), e2s[0] = 0
  static constexpr int BE = E2 + D;                              // [D] beta of reflector k
  static constexpr int WV = BE + D;                              // [D] w of the current step
  static constexpr int LAM = WV + D;                             // [RP] eigenvalues of T
  static constexpr int TH = LAM + RP;                            // [RP] Rayleigh quotients
  static constexpr int RH = TH + RP;                             // [RP] squared residual norms
  static constexpr int SG = RH + RP;                             // [RP] gauge signs
  static constexpr int PART = SG + RP;                           // [NW][RP] per-warp partial sums
  static constexpr int TRI_FLOATS = PART + C::NW * RP;
  static constexpr int FLOATS = TRI_FLOATS > full_jacobi_floats<D>() ? TRI_FLOATS : full_jacobi_floats<D>();
  static constexpr size_t BYTES = (size_t)FLOATS * sizeof(float);
  static_assert(DG % 4 == 0 && EO % 4 == 0 && E2 % 4 == 0 && WV % 4 == 0 && EM % 4 == 0 && WORK % 4 == 0 &&
                VS % 4 == 0, "16-byte alignment of the regions");
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
__device__ __forceinline__ float pick4(const float4& v, int c) {
  return c == 0 ? v.x : c == 1 ? v.y : c == 2 ? v.z : v.w;
}
__device__ __forceinline__ void put4(float4& v, int c, float x) {
  if (c == 0) v.x = x; else if (c == 1) v.y = x; else if (c == 2) v.z = x; else v.w = x;
}

// Acceptance thresholds (chosen by the storage type).
struct TriTol {
  float eps_vec;     // bound on sin(angle) of a kept vector implied by its residual and gap
  float floor_rel;   // residuals below floor_rel * theta_1 are at the rounding level of fp32
  float ortho;       // largest |V^T V - I| entry that needs no further orthogonalisation
  float sweep_stop;  // of the Jacobi fallback
};

// Number of eigenvalues of T below x, for three values of x at once.  p_{i+1} = (d_i - x) p_i -
// e_{i-1}^2 p_{i-1} is the leading principal minor of order i+1 of T - x I; the sign changes
// along p_0 = 1, p_1, ..., p_D count the eigenvalues below x.  The off-diagonal squares are
// floored above zero, so an exact zero never persists, and an isolated zero gives one change
// whichever sign the hardware gives it.
template <int D>
__device__ __forceinline__ void sturm3(const float* __restrict__ dg, const float* __restrict__ e2s,
                                       float x0, float x1, float x2, int& c0, int& c1, int& c2) {
  float p0 = 1.f, p1 = 1.f, p2 = 1.f, q0 = 0.f, q1 = 0.f, q2 = 0.f;
  unsigned n0 = 0, n1 = 0, n2 = 0;
#pragma unroll 2
  for (int ib = 0; ib < D / 4; ++ib) {
    const float4 d4 = *reinterpret_cast<const float4*>(dg + 4 * ib);
    const float4 e4 = *reinterpret_cast<const float4*>(e2s + 4 * ib);
    const float dd[4] = {d4.x, d4.y, d4.z, d4.w}, ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float t0 = ee[u] * q0, t1 = ee[u] * q1, t2 = ee[u] * q2;
      const float r0 = fmaf(dd[u] - x0, p0, -t0);
      const float r1 = fmaf(dd[u] - x1, p1, -t1);
      const float r2 = fmaf(dd[u] - x2, p2, -t2);
      n0 += (__float_as_uint(r0) ^ __float_as_uint(p0)) >> 31;
      n1 += (__float_as_uint(r1) ^ __float_as_uint(p1)) >> 31;
      n2 += (__float_as_uint(r2) ^ __float_as_uint(p2)) >> 31;
      q0 = p0; p0 = r0; q1 = p1; p1 = r1; q2 = p2; p2 = r2;
    }
    // bring the larger of (p, q) back into [1, 2): |d - x| and e^2 are bounded by the scaling of G,
    // so four steps can neither overflow nor (factors above 2^-23 each) underflow
    const unsigned m0 = __float_as_uint(fmaxf(fabsf(p0), fabsf(q0))) >> 23;
    const unsigned m1 = __float_as_uint(fmaxf(fabsf(p1), fabsf(q1))) >> 23;
    const unsigned m2 = __float_as_uint(fmaxf(fabsf(p2), fabsf(q2))) >> 23;
    const float s0 = __uint_as_float((254u - m0) << 23), s1 = __uint_as_float((254u - m1) << 23);
    const float s2 = __uint_as_float((254u - m2) << 23);
    p0 *= s0; q0 *= s0; p1 *= s1; q1 *= s1; p2 *= s2; q2 *= s2;
  }
  c0 = (int)n0; c1 = (int)n1; c2 = (int)n2;
}

template <int D, int RP>
__global__ void __launch_bounds__(TriCfg<D>::NT, 1)
eig_tridiag_kernel(const float* __restrict__ gpart, const int* __restrict__ gram_status, int splits,
                   float* __restrict__ gsum, int r, int route, int sweep_cap, TriTol tol,
                   float* __restrict__ S, float* __restrict__ V, int* __restrict__ info,
                   int* __restrict__ route_taken) {
  using Cfg = TriCfg<D>;
  using L = TriSmem<D, RP>;
  constexpr int NT = Cfg::NT, NW = Cfg::NW, TW = Cfg::TW, RPL = Cfg::RPL, LD = Cfg::LD, NB = Cfg::NB;
  constexpr int NE = RP / 32;                 // eigenvalues (columns) per lane in the column-parallel phases
  extern __shared__ __align__(16) float smem[];
  float* hv = smem + L::HV;
  float* vs = smem + L::VS;
  float* work = smem + L::WORK;
  float* Em = smem + L::EM;
  float* dg = smem + L::DG;
  float* eo = smem + L::EO;
  float* e2s = smem + L::E2;
  float* betas = smem + L::BE;
  float* wv = smem + L::WV;
  float* lamv = smem + L::LAM;
  float* theta = smem + L::TH;
  float* rho2 = smem + L::RH;
  float* sgn = smem + L::SG;
  float* part = smem + L::PART;
  __shared__ float s_gmax, s_lo, s_hi, s_emax, s_trT;
  __shared__ double s_trace;
  __shared__ float s_red[2][4];
  __shared__ float s_scal[2];
  __shared__ int s_flags[4];
  __shared__ int s_why;

  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();          // everything below reads what the Gram kernel wrote

  // ---- 1. G = sum of the slices' partial Grams, in a fixed order -----------------------------
  float* Gs = work;    // [D][LD] staging copy
  float* gout = gsum + (size_t)b * D * D;
  {
    const float4* gp = reinterpret_cast<const float4*>(gpart + (size_t)b * splits * D * D);
    int lost = 0;
    for (int s = tid; s < splits; s += NT) lost |= (gram_status[b * splits + s] != kGramStatusOk);
    int bad = 0;
    for (int e = tid; e < D * D / 4; e += NT) {
      // fp32 sums in a fixed order (GW slices at a time, pairwise within the group); all loads of a
      // group are issued before the first add: the loop is bound by their latency
      constexpr int GW = 16;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s = 0; s < splits; s += GW) {
        float4 v[GW];
#pragma unroll
        for (int u = 0; u < GW; ++u)
          v[u] = (s + u < splits) ? __ldg(gp + (size_t)(s + u) * (D * D / 4) + e)
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
      *reinterpret_cast<float4*>(Gs + (e / (D / 4)) * LD + (e % (D / 4)) * 4) = acc;
      reinterpret_cast<float4*>(gout)[e] = acc;      // the residual check and the fallback read it back
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
      return;
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
    if (warp < TW) {
      float a[RPL][D];
      int rowq[RPL];
#pragma unroll
      for (int q = 0; q < RPL; ++q) {
        rowq[q] = (TW == 1) ? lane + 32 * q : warp * 32 + lane;
#pragma unroll
        for (int jb = 0; jb < NB; ++jb) {
          const float4 g = *reinterpret_cast<const float4*>(Gs + rowq[q] * LD + 4 * jb);
          a[q][4 * jb] = g.x * sc; a[q][4 * jb + 1] = g.y * sc;
          a[q][4 * jb + 2] = g.z * sc; a[q][4 * jb + 3] = g.w * sc;
        }
      }
      float xf[RPL];           // column k of the current matrix at my rows
#pragma unroll
      for (int q = 0; q < RPL; ++q) xf[q] = a[q][0];

      for (int k = 0; k < D - 2; ++k) {
        const int k1 = k + 1, jb0 = k1 >> 2, c1 = k1 & 3;
        const bool skip0 = (RPL == 2) && (k >= 32);      // the lanes' first rows are all done
        // x = column k below the subdiagonal; published as the reflector's vector (its element
        // k+1 is patched in by the readers once alpha is known)
        float xs[RPL], sq = 0.f;
#pragma unroll
        for (int q = 0; q < RPL; ++q) {
          xs[q] = rowq[q] > k1 ? xf[q] : 0.f;
          sq = fmaf(xs[q], xs[q], sq);
          hv[k * D + rowq[q]] = xs[q];
        }
        float tail2, x1, dk;
        if (TW == 1) {
          float cand1 = xf[0], candk = xf[0];
          if (RPL == 2) { cand1 = (k1 >= 32) ? xf[RPL - 1] : xf[0]; candk = (k >= 32) ? xf[RPL - 1] : xf[0]; }
          x1 = __shfl_sync(kFull, cand1, k1 & 31);
          dk = __shfl_sync(kFull, candk, k & 31);
          tail2 = warp_sum(sq);
          __syncwarp();
        } else {
          sq = warp_sum(sq);
          if (lane == 0) s_red[0][warp] = sq;
          if (rowq[0] == k1) s_scal[0] = xf[0];
          if (rowq[0] == k) s_scal[1] = xf[0];
          bar_named(1, TW * 32);
          tail2 = (s_red[0][0] + s_red[0][1]) + (s_red[0][2] + s_red[0][3]);
          x1 = s_scal[0]; dk = s_scal[1];
        }
        const bool reflect = tail2 > 1e-35f;               // uniform over the taking-part warps
        float alpha = x1, beta = 0.f, vk1 = 0.f;
        if (reflect) {
          const float nrm = sqrtf(fmaf(x1, x1, tail2));
          alpha = -copysignf(nrm, x1);
          vk1 = x1 - alpha;
          beta = 1.f / (nrm * (nrm + fabsf(x1)));
        }
        if (tid == 0) { dg[k] = dk; eo[k] = alpha; betas[k] = beta; }
        if (!reflect) {
          // nothing to annihilate: T takes the column as it is, the matrix stays
#pragma unroll
          for (int jb = 0; jb < NB; ++jb)
            if (jb == jb0) {
#pragma unroll
              for (int q = 0; q < RPL; ++q)
                xf[q] = c1 == 0 ? a[q][4 * jb] : c1 == 1 ? a[q][4 * jb + 1] : c1 == 2 ? a[q][4 * jb + 2] : a[q][4 * jb + 3];
            }
          if (TW > 1) bar_named(1, TW * 32);               // the exchange words are rewritten next step
          continue;
        }
        float vi[RPL];
#pragma unroll
        for (int q = 0; q < RPL; ++q) {
          vi[q] = (rowq[q] == k1) ? vk1 : xs[q];
          if (rowq[q] == k1) hv[k * D + k1] = vk1;          // the complete vector, for step 5
        }
        // p = beta * A v over the trailing block (lane-local: a row against the broadcast v)
        const float4* v4p = reinterpret_cast<const float4*>(hv + k * D);
        float pa[RPL][2];
#pragma unroll
        for (int q = 0; q < RPL; ++q) { pa[q][0] = 0.f; pa[q][1] = 0.f; }
#pragma unroll
        for (int jb = 0; jb < NB; ++jb)
          if (jb >= jb0) {
            float4 v4 = v4p[jb];
            if (jb == jb0) put4(v4, c1, vk1);
#pragma unroll
            for (int q = 0; q < RPL; ++q) {
              if (q == 0 && skip0) continue;
              float acc = pa[q][jb & 1];
              acc = fmaf(a[q][4 * jb], v4.x, acc);     acc = fmaf(a[q][4 * jb + 1], v4.y, acc);
              acc = fmaf(a[q][4 * jb + 2], v4.z, acc); acc = fmaf(a[q][4 * jb + 3], v4.w, acc);
              pa[q][jb & 1] = acc;
            }
          }
        float pi[RPL], pv = 0.f;
#pragma unroll
        for (int q = 0; q < RPL; ++q) {
          pi[q] = rowq[q] > k ? beta * (pa[q][0] + pa[q][1]) : 0.f;
          pv = fmaf(pi[q], vi[q], pv);
        }
        if (TW == 1) {
          pv = warp_sum(pv);
        } else {
          pv = warp_sum(pv);
          if (lane == 0) s_red[1][warp] = pv;
          bar_named(1, TW * 32);
          pv = (s_red[1][0] + s_red[1][1]) + (s_red[1][2] + s_red[1][3]);
        }
        const float kk = 0.5f * beta * pv;
        float wi[RPL];
#pragma unroll
        for (int q = 0; q < RPL; ++q) {
          wi[q] = fmaf(-kk, vi[q], pi[q]);
          wv[rowq[q]] = wi[q];
        }
        if (TW == 1) __syncwarp(); else bar_named(1, TW * 32);
        // A <- A - v w^T - w v^T on the trailing block; the first block touched holds column k+1
        const float4* w4p = reinterpret_cast<const float4*>(wv);
#pragma unroll
        for (int jb = 0; jb < NB; ++jb)
          if (jb >= jb0) {
            float4 v4 = v4p[jb];
            if (jb == jb0) put4(v4, c1, vk1);
            const float4 w4 = w4p[jb];
#pragma unroll
            for (int q = 0; q < RPL; ++q) {
              if (q == 0 && skip0) continue;
              a[q][4 * jb]     = fmaf(-vi[q], w4.x, fmaf(-wi[q], v4.x, a[q][4 * jb]));
              a[q][4 * jb + 1] = fmaf(-vi[q], w4.y, fmaf(-wi[q], v4.y, a[q][4 * jb + 1]));
              a[q][4 * jb + 2] = fmaf(-vi[q], w4.z, fmaf(-wi[q], v4.z, a[q][4 * jb + 2]));
              a[q][4 * jb + 3] = fmaf(-vi[q], w4.w, fmaf(-wi[q], v4.w, a[q][4 * jb + 3]));
              if (jb == jb0)
                xf[q] = c1 == 0 ? a[q][4 * jb] : c1 == 1 ? a[q][4 * jb + 1] : c1 == 2 ? a[q][4 * jb + 2] : a[q][4 * jb + 3];
            }
          }
      }
      // the last 2 x 2 block: xf holds column D-2
#pragma unroll
      for (int q = 0; q < RPL; ++q) {
        if (rowq[q] == D - 2) dg[D - 2] = xf[q];
        if (rowq[q] == D - 1) { eo[D - 2] = xf[q]; dg[D - 1] = a[q][D - 1]; }
      }
      if (tid == 0) { eo[D - 1] = 0.f; betas[D - 2] = 0.f; betas[D - 1] = 0.f; }
    }
    __syncthreads();

    // ---- 3. Gershgorin interval, floored squares, trace; multisection --------------------------
    if (warp == 0) {
      float lo = 3.0e38f, hi = -3.0e38f, tr = 0.f;
      for (int i = lane; i < D; i += 32) {
        const float rad = fabsf(eo[i]) + (i > 0 ? fabsf(eo[i - 1]) : 0.f);   // eo[D-1] = 0
        lo = fminf(lo, dg[i] - rad); hi = fmaxf(hi, dg[i] + rad);
        tr += dg[i];
      }
      lo = -warp_max(-lo); hi = warp_max(hi); tr = warp_sum(tr);
      const float tn = fmaxf(fabsf(lo), fabsf(hi));
      const float fl = (tn * 1.4901161e-08f) * (tn * 1.4901161e-08f);         // (2^-26 |T|)^2
      for (int i = lane; i < D; i += 32) e2s[i] = i > 0 ? fmaxf(eo[i - 1] * eo[i - 1], fl) : 0.f;
      if (lane == 0) {
        const float span = hi - lo;
        s_lo = lo - 1e-6f * span - 1e-30f; s_hi = hi + 1e-6f * span + 1e-30f; s_trT = tr;
      }
    }
    __syncthreads();
    const float tnorm = fmaxf(fabsf(s_lo), fabsf(s_hi));
    if (warp < NE) {
      const int j = warp * 32 + lane, jj = j < r ? j : r - 1;
      const int target = D - 1 - jj;      // lambda_(jj-th largest) >= x  <=>  #(eigenvalues < x) <= target
      float lo = s_lo, hi = s_hi;
#pragma unroll 1
      for (int step = 0; step < 13; ++step) {
        const float w = hi - lo;
        const float m1 = fmaf(0.25f, w, lo), m2 = fmaf(0.5f, w, lo), m3 = fmaf(0.75f, w, lo);
        int c1, c2, c3;
        sturm3<D>(dg, e2s, m1, m2, m3, c1, c2, c3);
        if (c1 > target) { hi = m1; }
        else if (c2 > target) { lo = m1; hi = m2; }
        else if (c3 > target) { lo = m2; hi = m3; }
        else { lo = m3; }
      }
      const float lam = 0.5f * (lo + hi);
      lamv[j] = lam;

      // ---- 4. twisted factorisation: one vector per lane -----------------------------------------
      float* tf = work;                 // [D][RP] forward pivots, then the upward multipliers
      float* tb = work + D * RP;        // [D][RP] backward pivots, then the downward multipliers
      const float pfl = tnorm * 9.3132257e-10f;                              // pivot floor 2^-30 |T|
      {
        float qf = dg[0] - lam, qb = dg[D - 1] - lam;
        qf = fabsf(qf) < pfl ? -pfl : qf; qb = fabsf(qb) < pfl ? -pfl : qb;
        tf[j] = qf; tb[(D - 1) * RP + j] = qb;
#pragma unroll 4
        for (int t = 1; t < D; ++t) {
          const int ib = D - 1 - t;
          qf = (dg[t] - lam) - __fdividef(e2s[t], qf);
          qb = (dg[ib] - lam) - __fdividef(e2s[ib + 1], qb);
          qf = fabsf(qf) < pfl ? -pfl : qf; qb = fabsf(qb) < pfl ? -pfl : qb;
          tf[t * RP + j] = qf; tb[ib * RP + j] = qb;
        }
      }
      int kt = 0;
      {
        float best = 3.0e38f;
#pragma unroll 4
        for (int i = 0; i < D; ++i) {
          const float qf = tf[i * RP + j], qb = tb[i * RP + j];
          const float gam = fabsf((qf + qb) - (dg[i] - lam));
          if (gam < best) { best = gam; kt = i; }
          // z_i = -(e_i / q+_i) z_{i+1} going up, z_i = -(e_{i-1} / q-_i) z_{i-1} going down
          tf[i * RP + j] = -__fdividef(eo[i], qf);
          tb[i * RP + j] = i > 0 ? -__fdividef(eo[i - 1], qb) : 0.f;
        }
      }
      float ss = 1.f;
      {
        float zu = 1.f, zd = 1.f;
#pragma unroll 4
        for (int t = 1; t < D; ++t) {
          const int iu = D - 1 - t;            // upward: D-2 .. 0;  downward: 1 .. D-1
          const float mu = tf[iu * RP + j], md = tb[t * RP + j];
          if (iu < kt) { zu *= mu; ss = fmaf(zu, zu, ss); }
          if (t > kt) { zd *= md; ss = fmaf(zd, zd, ss); }
          if (iu < kt) vs[iu * RP + j] = zu;
          if (t > kt) vs[t * RP + j] = zd;
        }
        vs[kt * RP + j] = 1.f;
      }
      const float zn = rsqrtf(ss);

      // ---- 5. back-transformation: v = H_0 H_1 ... H_{D-3} z, the vector in registers -------------
      float z[D];
#pragma unroll
      for (int i = 0; i < D; ++i) z[i] = vs[i * RP + j] * zn;
#pragma unroll 1
      for (int k = D - 3; k >= 0; --k) {
        const float beta = betas[k];
        if (beta == 0.f) continue;                      // uniform
        const int ib0 = (k + 1) >> 2;                   // rows <= k of reflector k are zero
        const float4* h4 = reinterpret_cast<const float4*>(hv + k * D);
        float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
        for (int ib = 0; ib < NB; ++ib)
          if (ib >= ib0) {
            const float4 h = h4[ib];
            d0 = fmaf(h.x, z[4 * ib], d0); d1 = fmaf(h.y, z[4 * ib + 1], d1);
            d2 = fmaf(h.z, z[4 * ib + 2], d2); d3 = fmaf(h.w, z[4 * ib + 3], d3);
          }
        const float c = -beta * ((d0 + d1) + (d2 + d3));
#pragma unroll
        for (int ib = 0; ib < NB; ++ib)
          if (ib >= ib0) {
            const float4 h = h4[ib];
            z[4 * ib] = fmaf(c, h.x, z[4 * ib]);         z[4 * ib + 1] = fmaf(c, h.y, z[4 * ib + 1]);
            z[4 * ib + 2] = fmaf(c, h.z, z[4 * ib + 2]); z[4 * ib + 3] = fmaf(c, h.w, z[4 * ib + 3]);
          }
      }
#pragma unroll
      for (int i = 0; i < D; ++i) vs[i * RP + j] = z[i];
    }
    __syncthreads();
    pdl_trigger();     // the long serial part is over: the next kernel may start launching

    // G back into shared memory (over the reflectors), for the residuals
    float* Gsm = hv;   // [D][D], sc * G
    for (int e = tid; e < D * D / 4; e += NT) {
      float4 g = reinterpret_cast<const float4*>(gout)[e];
      g.x *= sc; g.y *= sc; g.z *= sc; g.w *= sc;
      reinterpret_cast<float4*>(Gsm)[e] = g;
    }

    // ---- 6. V <- V (I - (V^T V - I) / 2) while V^T V - I is above the rounding level -----------
    // Column-parallel: lane = column(s) c, c + 32; a warp takes RP / NW rows a of E.
    constexpr int AW = RP / NW;
    float* Vc = vs;        // current vectors
    float* Vn = work;      // next (the twisted-factorisation buffers are free now)
    for (;;) {
      float acc[NE][AW];
#pragma unroll
      for (int h = 0; h < NE; ++h)
#pragma unroll
        for (int u = 0; u < AW; ++u) acc[h][u] = 0.f;
      const int a0 = warp * AW;
#pragma unroll 2
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
      if (passes == 3 || !(em <= 0.25f)) { ok = false; if (tid == 0) s_why |= kWhyOrtho; break; }
      ++passes;
      // rows i of V' for this warp: D / NW of them; lane = column(s)
      float ecol[NE][RP];
#pragma unroll
      for (int h = 0; h < NE; ++h)
#pragma unroll
        for (int a = 0; a < RP; ++a) ecol[h][a] = Em[a * RP + 32 * h + lane];
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
          Vn[i * RP + 32 * h + lane] = fmaf(-0.5f, o[h], Vc[i * RP + 32 * h + lane]);
      }
      __syncthreads();
      float* t = Vc; Vc = Vn; Vn = t;
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
#pragma unroll 1
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

    if (ok || route == kRouteTridiag) {
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
        if (tid < r) S[(size_t)b * r + tid] = sqrtf(fmaxf(m, 0.f) / sc);
      }
      __syncthreads();
      for (int e = tid; e < D * r; e += NT) {
        const int i = e / r, j = e % r;
        V[(size_t)b * D * r + e] = Vc[i * RP + j] * sgn[j];
      }
      if (tid == 0) {
        if (info) info[b] = ok ? 0 : SOLAR_INFO_NOT_CERTIFIED;
        if (route_taken) route_taken[b] = kRouteTridiag | (passes << 16) | (s_why << 24);
      }
      return;
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
}

template <int D, int RP>
cudaError_t launch_tri(int B, int r, int route, int sweep_cap, TriTol tol, const float* gpart,
                       const int* gram_status, int splits, float* gsum, float* S, float* V, int* info,
                       int* route_taken, cudaStream_t st) {
  using L = TriSmem<D, RP>;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_set[dev]) {
    e = cudaFuncSetAttribute(eig_tridiag_kernel<D, RP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)L::BYTES);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_set[dev] = true;
  }
  return launch_pdl(eig_tridiag_kernel<D, RP>, dim3(B), dim3(TriCfg<D>::NT), L::BYTES, st, gpart, gram_status,
                    splits, gsum, r, route, sweep_cap, tol, S, V, info, route_taken);
}

}  // namespace

cudaError_t launch_eig_tridiag(int B, int d, int r, solar_dtype_t dt, int route, int sweep_cap,
                               const float* gpart, const int* gram_status, int splits, float* gsum,
                               float* S, float* V, int* info, int* route_taken, cudaStream_t st) {
  TriTol tol;
  if (dt == SOLAR_BF16) {
    tol.eps_vec = 1e-3f; tol.floor_rel = 64.f * kUnit; tol.ortho = 4e-6f; tol.sweep_stop = 1e-3f;
  } else {
    tol.eps_vec = 1e-5f; tol.floor_rel = 32.f * kUnit; tol.ortho = 2e-6f; tol.sweep_stop = 1e-5f;
  }
  const bool wide = r > 32;
  switch (d) {
    case 32:
      return launch_tri<32, 32>(B, r, route, sweep_cap, tol, gpart, gram_status, splits, gsum, S, V, info, route_taken, st);
    case 64:
      return wide ? launch_tri<64, 64>(B, r, route, sweep_cap, tol, gpart, gram_status, splits, gsum, S, V, info, route_taken, st)
                  : launch_tri<64, 32>(B, r, route, sweep_cap, tol, gpart, gram_status, splits, gsum, S, V, info, route_taken, st);
    case 128:
      return wide ? launch_tri<128, 64>(B, r, route, sweep_cap, tol, gpart, gram_status, splits, gsum, S, V, info, route_taken, st)
                  : launch_tri<128, 32>(B, r, route, sweep_cap, tol, gpart, gram_status, splits, gsum, S, V, info, route_taken, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace solar
