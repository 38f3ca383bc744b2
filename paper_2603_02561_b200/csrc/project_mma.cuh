// Factor-token projections of Eq. 11 on the tensor cores, for bf16 weights and d = 64 or 128:
//   Key_r   = (V Sigma)^T W_K   [r,d]
//   Value_r = (V Sigma)^T W_V   [r,d]
//   T       = scale * W_Q Key_r^T  [d,r]   (so that the scores of Eq. 12 are C T)
// written as the attention kernels' packed operands (T^T and Value_r^T, each as a high and a
// low bf16 half) and, on request, as fp32 copies.  Three small GEMMs per user -- far too small
// for tcgen05 (M would be 16 or 32) -- so they run as warp-level mma.sync.m16n8k16 with fp32
// accumulation: the fp32 factor V Sigma enters as a high and a low bf16 half (two MMAs per
// product, ~16 mantissa bits), the weights are bf16 already, and Key_r never leaves the
// registers: the accumulator fragment of the first GEMM has the layout of the second GEMM's A
// fragment.  One job = (16 tokens) x (Key -> T | Value); the CTA's warps share the jobs.
// Included by the eigensolver (as the epilogue of a user's CTA) and by the stand-alone
// projection kernel, so both produce the same bits.
#pragma once

#include <cuda_bf16.h>

#include "solar_internal.cuh"

namespace solar {
namespace pmma {

// Shared-memory layout in bytes for rp16 = 16 ceil(r / 16) token rows.  The fp32 factor
// [D][rp] (rp = r rounded up to 4) is expected at offset 0.
template <int D> struct Lay {
  static constexpr int P = (D + 8) * 2;                 // row pitch of the k-contiguous bf16 arrays: conflict-free
  __host__ __device__ static constexpr int vsh(int rp16) { return D * rp16 * 4; }          // [rp16][D+8] high halves of (V Sigma)^T
  __host__ __device__ static constexpr int vsl(int rp16) { return vsh(rp16) + rp16 * P; }  // low halves
  __host__ __device__ static constexpr int wk(int rp16) { return vsl(rp16) + rp16 * P; }   // [D][D+8] W_K as stored
  __host__ __device__ static constexpr int wq(int rp16) { return wk(rp16) + D * P; }
  __host__ __device__ static constexpr int wv(int rp16) { return wq(rp16) + D * P; }
  __host__ __device__ static constexpr int vout(int rp16) { return wv(rp16) + D * P; }     // [2][D][rp16+8] Value_r^T halves
  __host__ __device__ static constexpr int bytes(int rp16) { return vout(rp16) + 2 * D * (rp16 + 8) * 2; }
};

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
// (a, b) as a pair of high halves and the pair of what they leave over
__device__ __forceinline__ void split2(float a, float b, uint32_t& hi, uint32_t& lo) {
  const float ah = __bfloat162float(__float2bfloat16_rn(a)), bh = __bfloat162float(__float2bfloat16_rn(b));
  hi = pack2(ah, bh);
  lo = pack2(a - ah, b - bh);
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Four 8x8 bf16 blocks, transposed on the way: B fragments (pairs along k) from a matrix stored
// with k along the rows.
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&x)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3])
               : "r"((uint32_t)__cvta_generic_to_shared(p)));
}

// Every thread of the CTA (NT threads) calls this after a barrier behind the writes of the fp32
// factor at sm[0 ..).  pad_to: token slots to leave zero-filled in the packed operands
// (>= 16 ceil(r / 16), <= kTokenSlots).  Tf / Vr: fp32 copies T [D][r] and Value_r [r][D], or
// both nullptr.
template <int D, int NT>
__device__ __forceinline__ void project(unsigned char* __restrict__ sm, int r, const void* __restrict__ Wq,
                                        const void* __restrict__ Wk, const void* __restrict__ Wv, float scale,
                                        __nv_bfloat16* __restrict__ Tpk, __nv_bfloat16* __restrict__ Vpk,
                                        float* __restrict__ Tf, float* __restrict__ Vr, int pad_to, int tid) {
  using L = Lay<D>;
  constexpr int P = L::P, NW = NT / 32, KS = D / 16, NTL = D / 8;
  const int rp = (r + 3) & ~3, rp16 = (r + 15) & ~15, mt_n = rp16 / 16;
  const float* VS = reinterpret_cast<const float*>(sm);
  unsigned char* vsh = sm + L::vsh(rp16);
  unsigned char* vsl = sm + L::vsl(rp16);
  unsigned char* wks = sm + L::wk(rp16);
  unsigned char* wqs = sm + L::wq(rp16);
  unsigned char* wvs = sm + L::wv(rp16);
  unsigned char* vout = sm + L::vout(rp16);
  const int lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;

  // the three weights as they are stored (16-byte pieces; all loads of a thread first)
  {
    constexpr int NV = D * D / 8 / NT;
    static_assert(NV * NT * 8 == D * D, "whole pieces");
    uint4 raw[3][NV];
#pragma unroll
    for (int n = 0; n < NV; ++n) {
      raw[0][n] = __ldg(static_cast<const uint4*>(Wk) + tid + n * NT);
      raw[1][n] = __ldg(static_cast<const uint4*>(Wq) + tid + n * NT);
      raw[2][n] = __ldg(static_cast<const uint4*>(Wv) + tid + n * NT);
    }
#pragma unroll
    for (int n = 0; n < NV; ++n) {
      const int v = tid + n * NT, row = v / (D / 8), c = v % (D / 8);
      *reinterpret_cast<uint4*>(wks + row * P + c * 16) = raw[0][n];
      *reinterpret_cast<uint4*>(wqs + row * P + c * 16) = raw[1][n];
      *reinterpret_cast<uint4*>(wvs + row * P + c * 16) = raw[2][n];
    }
  }
  // (V Sigma)^T as bf16 halves, token-major; token rows >= rp are zero rows
  for (int e = tid; e < rp16 * (D / 2); e += NT) {
    const int i = e % rp16, kp = e / rp16;
    const float a = i < rp ? VS[(2 * kp) * rp + i] : 0.f, c = i < rp ? VS[(2 * kp + 1) * rp + i] : 0.f;
    uint32_t hi, lo;
    split2(a, c, hi, lo);
    *reinterpret_cast<uint32_t*>(vsh + i * P + kp * 4) = hi;
    *reinterpret_cast<uint32_t*>(vsl + i * P + kp * 4) = lo;
  }
  // token slots rp16 .. pad_to - 1 of the packed operands stay zero
  {
    const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);
    const int extra = pad_to - rp16;
    for (int e = tid; e < 2 * extra * (D / 8); e += NT) {
      const int h = e / (extra * (D / 8)), rem = e % (extra * (D / 8));
      reinterpret_cast<uint4*>(Tpk + ((size_t)h * kTokenSlots + rp16) * D)[rem] = z4;
    }
    for (int e = tid; e < 2 * D * (extra / 8); e += NT) {
      const int row = e / (extra / 8), c = e % (extra / 8);
      reinterpret_cast<uint4*>(Vpk + (size_t)row * kTokenSlots + rp16)[c] = z4;      // row runs over [2][D]
    }
  }
  __syncthreads();

  for (int job = warp; job < 2 * mt_n; job += NW) {
    const int mt = job % mt_n, kind = job / mt_n;          // kind 0: Key_r, then T; 1: Value_r
    const int i0 = 16 * mt + g;                            // this lane's token rows: i0 and i0 + 8
    // A fragments of (V Sigma)^T for all k
    uint32_t ah[KS][4], al[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int o0 = i0 * P + (16 * ks + 2 * t) * 2, o1 = o0 + 8 * P;
      ah[ks][0] = *reinterpret_cast<const uint32_t*>(vsh + o0);
      ah[ks][1] = *reinterpret_cast<const uint32_t*>(vsh + o1);
      ah[ks][2] = *reinterpret_cast<const uint32_t*>(vsh + o0 + 16);
      ah[ks][3] = *reinterpret_cast<const uint32_t*>(vsh + o1 + 16);
      al[ks][0] = *reinterpret_cast<const uint32_t*>(vsl + o0);
      al[ks][1] = *reinterpret_cast<const uint32_t*>(vsl + o1);
      al[ks][2] = *reinterpret_cast<const uint32_t*>(vsl + o0 + 16);
      al[ks][3] = *reinterpret_cast<const uint32_t*>(vsl + o1 + 16);
    }
    // X[i][j] = sum_k (V Sigma)[k][i] W[k][j], all D columns j of the 16 tokens
    const unsigned char* wsrc = kind == 0 ? wks : wvs;
    float acc[NTL][4];
#pragma unroll
    for (int nt = 0; nt < NTL; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int nt = 0; nt < NTL; nt += 2) {
        uint32_t bfr[4];       // b0, b1 of column block nt; b0, b1 of block nt + 1
        ldsm_x4_trans(bfr, wsrc + (16 * ks + 8 * ((lane >> 3) & 1) + (lane & 7)) * P + (8 * (nt + (lane >> 4))) * 2);
        mma16816(acc[nt], ah[ks], bfr[0], bfr[1]);
        mma16816(acc[nt], al[ks], bfr[0], bfr[1]);
        mma16816(acc[nt + 1], ah[ks], bfr[2], bfr[3]);
        mma16816(acc[nt + 1], al[ks], bfr[2], bfr[3]);
      }
    }
    if (kind == 1) {
      // Value_r^T halves into the staging tile [h][j][token]; the fp32 copy straight from the registers
#pragma unroll
      for (int nt = 0; nt < NTL; ++nt) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int i = i0 + 8 * (q >> 1), j = 8 * nt + 2 * t + (q & 1);
          const float x = acc[nt][q];
          const __nv_bfloat16 hi = __float2bfloat16_rn(x);
          __nv_bfloat16* row = reinterpret_cast<__nv_bfloat16*>(vout) + (size_t)j * (rp16 + 8) + i;
          row[0] = hi;
          row[(size_t)D * (rp16 + 8)] = __float2bfloat16_rn(x - __bfloat162float(hi));
        }
        if (Vr != nullptr) {
          if (i0 < r) *reinterpret_cast<float2*>(Vr + (size_t)i0 * D + 8 * nt + 2 * t) = make_float2(acc[nt][0], acc[nt][1]);
          if (i0 + 8 < r) *reinterpret_cast<float2*>(Vr + (size_t)(i0 + 8) * D + 8 * nt + 2 * t) = make_float2(acc[nt][2], acc[nt][3]);
        }
      }
      continue;
    }
    // Key_r as the A operand of T^T[i][k] = scale * sum_j Key_r[i][j] W_Q[k][j]
    uint32_t kh[KS][4], kl[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      split2(acc[2 * ks][0], acc[2 * ks][1], kh[ks][0], kl[ks][0]);
      split2(acc[2 * ks][2], acc[2 * ks][3], kh[ks][1], kl[ks][1]);
      split2(acc[2 * ks + 1][0], acc[2 * ks + 1][1], kh[ks][2], kl[ks][2]);
      split2(acc[2 * ks + 1][2], acc[2 * ks + 1][3], kh[ks][3], kl[ks][3]);
    }
#pragma unroll
    for (int nt = 0; nt < NTL; ++nt) {
      float tc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const unsigned char* wrow = wqs + (8 * nt + g) * P + (16 * ks + 2 * t) * 2;     // W_Q[k = 8 nt + g][j ..]
        const uint32_t b0 = *reinterpret_cast<const uint32_t*>(wrow), b1 = *reinterpret_cast<const uint32_t*>(wrow + 16);
        mma16816(tc, kh[ks], b0, b1);
        mma16816(tc, kl[ks], b0, b1);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) tc[q] *= scale;
      const int k0 = 8 * nt + 2 * t;
      uint32_t hi, lo;
      split2(tc[0], tc[1], hi, lo);
      *reinterpret_cast<uint32_t*>(Tpk + (size_t)i0 * D + k0) = hi;
      *reinterpret_cast<uint32_t*>(Tpk + ((size_t)kTokenSlots + i0) * D + k0) = lo;
      split2(tc[2], tc[3], hi, lo);
      *reinterpret_cast<uint32_t*>(Tpk + (size_t)(i0 + 8) * D + k0) = hi;
      *reinterpret_cast<uint32_t*>(Tpk + ((size_t)kTokenSlots + i0 + 8) * D + k0) = lo;
      if (Tf != nullptr) {
        if (i0 < r) { Tf[(size_t)k0 * r + i0] = tc[0]; Tf[(size_t)(k0 + 1) * r + i0] = tc[1]; }
        if (i0 + 8 < r) { Tf[(size_t)k0 * r + i0 + 8] = tc[2]; Tf[(size_t)(k0 + 1) * r + i0 + 8] = tc[3]; }
      }
    }
  }
  __syncthreads();
  // Value_r^T out: 16-byte pieces of the rows [h][j][0 .. rp16)
  for (int e = tid; e < 2 * D * (rp16 / 8); e += NT) {
    const int row = e / (rp16 / 8), c = e % (rp16 / 8);                                  // row runs over [2][D]
    reinterpret_cast<uint4*>(Vpk + (size_t)row * kTokenSlots)[c] =
        *reinterpret_cast<const uint4*>(vout + ((size_t)row * (rp16 + 8) + 8 * c) * 2);
  }
}

}  // namespace pmma
}  // namespace solar
