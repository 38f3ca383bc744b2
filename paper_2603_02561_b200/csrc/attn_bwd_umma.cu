// Streaming kernel of the attention backward pass on the tensor cores (bf16 storage,
// d = 64 or 128).  With S = C T, P = softmax_r(S), O = P Value_r (Eq. 11-12 folded):
//   dP = dO Value_r^T,  dS = P o (dP - rowsum(P o dP)),
//   dC = dS T^T,   dT += C^T dS,   dValue_r^T += dO^T P      (the two sums run over M).
// One CTA per chunk of 128-row candidate tiles of one user.  Per tile:
//   TMA: C and dO tiles -> shared memory (128-byte swizzle; rows past M read as zero and
//        therefore add nothing to the sums)
//   tcgen05.mma: S = C T and dP = dO Value_r^T (high + low halves of the per-user operands)
//   tcgen05.ld: one row per thread; softmax and dS in registers; P and dS return to shared
//        memory as bf16 high/low halves
//   tcgen05.mma: dC = dS T^T (K-major operands);  dT += C^T dS and dValue_r^T += dO^T P with
//        the SAME shared-memory tiles read as MN-major operands (K = the 128 rows), both
//        accumulating in tensor memory across the tiles of the chunk
//   tcgen05.ld: dC -> bf16 -> shared memory -> TMA store
// At the end the two accumulators go to the chunk's partial in the workspace.  Scores and
// probabilities never leave the SM.  Every wait is bounded; if one runs out, the chunk's
// dC rows and its partial are written as NaN.
#include "sm100_ptx.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kRows = 128;
constexpr int kBoxBytes = kRows * 128;
constexpr int kErrOps = 0x51, kErrLoad = 0x52, kErrScores = 0x53, kErrOut = 0x54, kErrAcc = 0x55;
constexpr int kColS = 0, kColP = 64, kColT = 128, kColV = 192, kTmemCols = 256;

template <int D> struct BwdCfg {
  static constexpr int KB = D / 64;
  static constexpr int TILE_BYTES = KB * kBoxBytes;                 // C, dO, dC tiles
  __host__ __device__ static constexpr int tok_bytes(int np) { return 2 * KB * np * 128; }   // [2][KB][np][128 B]
  static constexpr int TK_BYTES = 2 * D * 128;                      // T hi/lo as [2][D rows][128 B]
  static constexpr int PD_BYTES = 2 * kBoxBytes;                    // P or dS, hi/lo
  static constexpr size_t smem(int np) {
    return (size_t)2 * TILE_BYTES + 2 * tok_bytes(np) + TK_BYTES + 2 * PD_BYTES + 1024;
  }
};

// eight values as a bf16 high half and the bf16 of what the high half misses
__device__ __forceinline__ void split8(const float* x, uint4& hi, uint4& lo) {
  uint32_t h[4], l[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float x0 = x[2 * q], x1 = x[2 * q + 1];
    const float h0 = __bfloat162float(__float2bfloat16_rn(x0));
    const float h1 = __bfloat162float(__float2bfloat16_rn(x1));
    h[q] = ptx::pack_bf16(h0, h1);
    l[q] = ptx::pack_bf16(x0 - h0, x1 - h1);
  }
  hi = make_uint4(h[0], h[1], h[2], h[3]);
  lo = make_uint4(l[0], l[1], l[2], l[3]);
}

template <int D>
__global__ void __launch_bounds__(128, 1)
attn_bwd_umma_kernel(const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmG,
                     const __grid_constant__ CUtensorMap tmDC, const __grid_constant__ CUtensorMap tmT,
                     const __grid_constant__ CUtensorMap tmVk, const __grid_constant__ CUtensorMap tmTk,
                     int r, unsigned flags, __nv_bfloat16* __restrict__ dC, float* __restrict__ part, int M,
                     int tiles_per_cta) {
  using Cfg = BwdCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int np = (r + 15) & ~15;
  const int tok_tile = np * 128;               // bytes of one [np rows][128 B] tile
  uint8_t* sC = base;                          // [KB][128][128 B]  candidates, then the dC tile
  uint8_t* sG = sC + Cfg::TILE_BYTES;          // [KB][128][128 B]  dO
  uint8_t* sT = sG + Cfg::TILE_BYTES;          // [2][KB][np][128 B]  T^T hi/lo       (B of S = C T)
  uint8_t* sVk = sT + Cfg::tok_bytes(np);      // [2][KB][np][128 B]  Value_r hi/lo   (B of dP = dO Value_r^T)
  uint8_t* sTk = sVk + Cfg::tok_bytes(np);     // [2][D][128 B]       T hi/lo         (B of dC = dS T^T)
  uint8_t* sP = sTk + Cfg::TK_BYTES;           // [2][128][128 B]     P hi/lo
  uint8_t* sD = sP + Cfg::PD_BYTES;            // [2][128][128 B]     dS hi/lo
  __shared__ __align__(8) uint64_t bar_ops, bar_load, bar_s, bar_o;
  __shared__ uint32_t s_tmem;
  __shared__ int s_err;

  const int b = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles = (M + kRows - 1) / kRows;
  const int t_begin = chunk * tiles_per_cta;
  const int t_end = min(tiles, t_begin + tiles_per_cta);

  if (tid == 0) {
    s_err = 0;
    ptx::mbar_init(&bar_ops, 1); ptx::mbar_init(&bar_load, 1); ptx::mbar_init(&bar_s, 1); ptx::mbar_init(&bar_o, 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmC); ptx::prefetch_tensormap(&tmG); ptx::prefetch_tensormap(&tmDC);
    ptx::prefetch_tensormap(&tmT); ptx::prefetch_tensormap(&tmVk); ptx::prefetch_tensormap(&tmTk);
  }
  if (warp == 1) ptx::tmem_alloc(&s_tmem, kTmemCols);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = s_tmem;
  volatile int* err = &s_err;
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  const bool use_softmax = !(flags & SOLAR_FLAG_NO_SOFTMAX);

  if (tid == 0) {
    // the per-user operands, once
    ptx::mbar_arrive_expect_tx(&bar_ops, 2 * Cfg::tok_bytes(np) + Cfg::TK_BYTES);
#pragma unroll
    for (int x = 0; x < Cfg::KB; ++x)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        ptx::tma_load_3d(sT + (h * Cfg::KB + x) * tok_tile, &tmT, &bar_ops, x * 64, h * kTokenSlots, b);
        ptx::tma_load_3d(sVk + (h * Cfg::KB + x) * tok_tile, &tmVk, &bar_ops, x * 64, h * kTokenSlots, b);
      }
#pragma unroll
    for (int h = 0; h < 2; ++h) ptx::tma_load_3d(sTk + h * (D * 128), &tmTk, &bar_ops, 0, h * D, b);
  }

  bool ops_ready = false;
  for (int t = t_begin; t < t_end; ++t) {
    const int it = t - t_begin;                // tile index within the chunk: barrier phases
    const int m0 = t * kRows;
    if (tid == 0) {
      ptx::tma_store_wait_read();              // the previous dC tile has left sC
      ptx::mbar_arrive_expect_tx(&bar_load, 2 * Cfg::TILE_BYTES);
#pragma unroll
      for (int x = 0; x < Cfg::KB; ++x) {
        ptx::tma_load_3d(sC + x * kBoxBytes, &tmC, &bar_load, x * 64, m0, b);
        ptx::tma_load_3d(sG + x * kBoxBytes, &tmG, &bar_load, x * 64, m0, b);
      }
    }
    if (tid == 32) {
      // ---- S = C T and dP = dO Value_r^T : M = 128, N = np, K = D, high + low halves ----
      bool ok = ops_ready || ptx::mbar_wait(&bar_ops, 0, err, kErrOps);
      ok = ok && ptx::mbar_wait(&bar_load, it & 1, err, kErrLoad);
      if (ok) {
        ptx::tc_fence_after_sync();
        const uint32_t idesc = ptx::umma_idesc_bf16(kRows, np, false, false);
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          const uint32_t abase = ptx::smem_u32(g == 0 ? sC : sG);
          const uint32_t bbase = ptx::smem_u32(g == 0 ? sT : sVk);
          bool acc = false;
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t a = abase + (kk / 4) * kBoxBytes + (kk % 4) * 32;
              const uint32_t bb = bbase + (h * Cfg::KB + kk / 4) * tok_tile + (kk % 4) * 32;
              ptx::umma_bf16_ss(tmem + (g == 0 ? kColS : kColP), ptx::umma_smem_desc(a, 0, 1024),
                                ptx::umma_smem_desc(bb, 0, 1024), idesc, acc);
              acc = true;
            }
        }
      }
      ptx::umma_commit(&bar_s);
    }
    ops_ready = true;
    __syncwarp();

    // ---- probabilities and dS, one candidate row per thread ---------------------------------
    const bool have_s = ptx::mbar_wait(&bar_s, it & 1, err, kErrScores);
    __syncwarp();
    ptx::tc_fence_after_sync();
    float p[kTokenSlots];
    {
      uint32_t v[32];
      ptx::tmem_ld_32x32(tmem + lane_base + kColS, v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) p[i] = __uint_as_float(v[i]);
      if (np > 32) {
        ptx::tmem_ld_32x32(tmem + lane_base + kColS + 32, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) p[32 + i] = __uint_as_float(v[i]);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) p[32 + i] = 0.f;
      }
    }
    float dot = 0.f;
    if (use_softmax) {
      float mx = -INFINITY;
#pragma unroll
      for (int i = 0; i < kTokenSlots; ++i) mx = (i < r) ? fmaxf(mx, p[i]) : mx;
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < kTokenSlots; ++i) {
        p[i] = (i < r) ? ptx::fast_exp2((p[i] - mx) * 1.4426950408889634f) : 0.f;
        sum += p[i];
      }
      const float inv = 1.f / sum;
#pragma unroll
      for (int i = 0; i < kTokenSlots; ++i) p[i] *= inv;
      // rowsum(P o dP): first pass over dP
#pragma unroll
      for (int c0 = 0; c0 < kTokenSlots; c0 += 32) {
        if (c0 < np) {
          uint32_t v[32];
          ptx::tmem_ld_32x32(tmem + lane_base + kColP + c0, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) dot = fmaf(p[c0 + i], __uint_as_float(v[i]), dot);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < kTokenSlots; ++i) p[i] = (i < r) ? p[i] : 0.f;
    }
    // second pass over dP: dS, and both matrices to shared memory as hi/lo halves
#pragma unroll
    for (int c0 = 0; c0 < kTokenSlots; c0 += 32) {
      if (c0 < np) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(tmem + lane_base + kColP + c0, v);
        ptx::tmem_ld_wait();
        float dsv[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float dp = __uint_as_float(v[i]);
          dsv[i] = use_softmax ? p[c0 + i] * (dp - dot) : ((c0 + i < r) ? dp : 0.f);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 hi, lo;
          split8(&p[c0 + 8 * c], hi, lo);
          *reinterpret_cast<uint4*>(sP + ptx::swz128(tid, c0 / 8 + c)) = hi;
          *reinterpret_cast<uint4*>(sP + kBoxBytes + ptx::swz128(tid, c0 / 8 + c)) = lo;
          split8(&dsv[8 * c], hi, lo);
          *reinterpret_cast<uint4*>(sD + ptx::swz128(tid, c0 / 8 + c)) = hi;
          *reinterpret_cast<uint4*>(sD + kBoxBytes + ptx::swz128(tid, c0 / 8 + c)) = lo;
        }
      }
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();

    if (tid == 32) {
      ptx::tc_fence_after_sync();
      if (have_s && *err == 0) {
        // ---- dC = dS T^T : M = 128, N = D, K = np; hi*hi + hi*lo + lo*hi ----------------
        {
          const uint32_t idesc = ptx::umma_idesc_bf16(kRows, D, false, false);
          bool acc = false;
#pragma unroll
          for (int term = 0; term < 3; ++term) {
            const uint32_t a = ptx::smem_u32(sD) + (term == 2 ? kBoxBytes : 0);
            const uint32_t bb = ptx::smem_u32(sTk) + (term == 1 ? D * 128 : 0);
            for (int kk = 0; kk < np / 16; ++kk) {
              ptx::umma_bf16_ss(tmem + kColS, ptx::umma_smem_desc(a + kk * 32, 0, 1024),
                                ptx::umma_smem_desc(bb + kk * 32, 0, 1024), idesc, acc);
              acc = true;
            }
          }
        }
        // ---- dT += C^T dS and dValue_r^T += dO^T P : M = D, N = np, K = the 128 rows ----------
        {
          const uint32_t idesc = ptx::umma_idesc_bf16(D, np, true, true);
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            const uint32_t abase = ptx::smem_u32(g == 0 ? sC : sG);
            const uint32_t bbase = ptx::smem_u32(g == 0 ? sD : sP);
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
              for (int ks = 0; ks < kRows / 16; ++ks) {
                // 16 rows = two 8-row swizzle atoms of 1024 B; 64-column boxes are kBoxBytes apart
                const uint64_t ad = ptx::umma_smem_desc(abase + ks * 2048, kBoxBytes, 1024);
                const uint64_t bd = ptx::umma_smem_desc(bbase + h * kBoxBytes + ks * 2048, kBoxBytes, 1024);
                ptx::umma_bf16_ss(tmem + (g == 0 ? kColT : kColV), ad, bd, idesc, (it | h | ks) != 0);
              }
          }
        }
      }
      ptx::umma_commit(&bar_o);
    }
    __syncwarp();

    // ---- dC tile: tensor memory -> bf16 -> shared memory (over the candidate tile) -> TMA ----
    ptx::mbar_wait(&bar_o, it & 1, err, kErrOut);
    __syncwarp();
    ptx::tc_fence_after_sync();
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t v[32];
      ptx::tmem_ld_32x32(tmem + lane_base + kColS + c0, v);
      ptx::tmem_ld_wait();
      uint8_t* box = sC + (c0 / 64) * kBoxBytes;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint4 w = make_uint4(
            ptx::pack_bf16(__uint_as_float(v[8 * c + 0]), __uint_as_float(v[8 * c + 1])),
            ptx::pack_bf16(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3])),
            ptx::pack_bf16(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5])),
            ptx::pack_bf16(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7])));
        *reinterpret_cast<uint4*>(box + ptx::swz128(tid, (c0 % 64) / 8 + c)) = w;
      }
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (s_err == 0) {
      if (tid == 0) {
#pragma unroll
        for (int x = 0; x < Cfg::KB; ++x) ptx::tma_store_3d(&tmDC, sC + x * kBoxBytes, x * 64, m0, b);
        ptx::tma_store_commit();
      }
    } else if (m0 + tid < M) {
      uint4* dst = reinterpret_cast<uint4*>(dC + ((size_t)b * M + m0 + tid) * D);
      const uint4 qnan = make_uint4(0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u);
#pragma unroll
      for (int c = 0; c < D / 8; ++c) dst[c] = qnan;
    }
    ptx::tc_fence_after_sync();
  }
  if (tid == 0) ptx::tma_store_wait_all();

  // ---- the chunk's partial: [2][D][64] fp32, columns >= np zero --------------------------------
  // (the last tile's wait on bar_o covered every MMA into the two accumulators)
  float* out = part + ((size_t)b * gridDim.x + chunk) * 2 * D * kTokenSlots;
  const bool good = (s_err == 0) && (t_end > t_begin);
  // M = 128: accumulator row k sits in lane k.  M = 64: rows 16q .. 16q+15 sit in lanes 32q .. 32q+15.
  const int row = (D == 128) ? (warp * 32 + lane) : (warp * 16 + lane);
  const bool has_row = (D == 128) || (lane < 16);
#pragma unroll
  for (int g = 0; g < 2; ++g) {
#pragma unroll
    for (int c0 = 0; c0 < kTokenSlots; c0 += 32) {
      uint32_t v[32];
      if (good && c0 < np) {
        ptx::tmem_ld_32x32(tmem + lane_base + (g == 0 ? kColT : kColV) + c0, v);
        ptx::tmem_ld_wait();
      } else {
        const uint32_t fill = (s_err != 0) ? 0x7fc00000u : 0u;
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = fill;
      }
      if (has_row) {
        float4* dst = reinterpret_cast<float4*>(out + ((size_t)g * D + row) * kTokenSlots + c0);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                               __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
      }
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, kTmemCols);
}

// T [d][r] and Value_r [r][d] (fp32, written by the prepare kernel) as the two extra bf16
// operand images of the kernel above: Tkm [2][d][64] (T, tokens along K, zero past r) and
// Vkm [2][64][d] (Value_r, zero rows past r), each as a high and a low half.
__global__ void attn_bwd_pack_kernel(const char* __restrict__ ws, AttnWs lay, int d, int r,
                                     __nv_bfloat16* __restrict__ pk) {
  const int b = blockIdx.y;
  const char* wsb = ws + (size_t)b * lay.per_user;
  const float* Tf = reinterpret_cast<const float*>(wsb + lay.tf_off);
  const float* Vr = reinterpret_cast<const float*>(wsb + lay.vr_off);
  __nv_bfloat16* Tkm = pk + (size_t)b * 4 * kTokenSlots * d;
  __nv_bfloat16* Vkm = Tkm + 2 * kTokenSlots * d;
  for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < d * kTokenSlots; e += gridDim.x * blockDim.x) {
    const int k = e / kTokenSlots, i = e % kTokenSlots;
    const float t = i < r ? Tf[k * r + i] : 0.f;
    const __nv_bfloat16 th = __float2bfloat16_rn(t);
    Tkm[e] = th;
    Tkm[d * kTokenSlots + e] = __float2bfloat16_rn(t - __bfloat162float(th));
    const int i2 = e / d, j = e % d;
    const float v = i2 < r ? Vr[i2 * d + j] : 0.f;
    const __nv_bfloat16 vh = __float2bfloat16_rn(v);
    Vkm[e] = vh;
    Vkm[kTokenSlots * d + e] = __float2bfloat16_rn(v - __bfloat162float(vh));
  }
}

template <int D>
cudaError_t launch_d(int B, int M, int r, const void* C, const void* dO, unsigned flags, void* dC, float* part,
                     __nv_bfloat16* pk, int tiles_per_cta, int chunks, const char* ws, const AttnWs& lay,
                     cudaStream_t st) {
  using Cfg = BwdCfg<D>;
  attn_bwd_pack_kernel<<<dim3(D * kTokenSlots / 256, B), 256, 0, st>>>(ws, lay, D, r, pk);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  CUtensorMap tmC, tmG, tmDC, tmT, tmVk, tmTk;
  const uint64_t pu = lay.per_user, pku = (uint64_t)4 * kTokenSlots * D * 2;
  const int np = (r + 15) & ~15;
  bool ok = encode_tmap_bf16_3d(&tmC, C, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmG, dO, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmDC, dC, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmT, ws + lay.tpk_off, D, 2 * kTokenSlots, (uint64_t)B, (uint64_t)D * 2, pu, 64, np);
  ok = ok && encode_tmap_bf16_3d(&tmTk, pk, kTokenSlots, 2 * D, (uint64_t)B, kTokenSlots * 2, pku, kTokenSlots, D);
  ok = ok && encode_tmap_bf16_3d(&tmVk, pk + 2 * kTokenSlots * D, D, 2 * kTokenSlots, (uint64_t)B, (uint64_t)D * 2, pku,
                                 64, np);
  if (!ok) return cudaErrorInvalidValue;
  e = cudaFuncSetAttribute(attn_bwd_umma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)Cfg::smem(kTokenSlots));
  if (e != cudaSuccess) return e;
  attn_bwd_umma_kernel<D><<<dim3(chunks, B), 128, Cfg::smem(np), st>>>(
      tmC, tmG, tmDC, tmT, tmVk, tmTk, r, flags, static_cast<__nv_bfloat16*>(dC), part, M, tiles_per_cta);
  return cudaGetLastError();
}

}  // namespace

bool attn_bwd_umma_supported(int M, int d, solar_dtype_t dt) {
  return dt == SOLAR_BF16 && (d == 64 || d == 128) && M >= 1;
}

cudaError_t launch_attn_bwd_umma(int B, int M, int d, int r, const void* C, const void* dO, unsigned flags,
                                 void* dC, float* part, void* pk, int tiles_per_cta, int chunks, const char* ws,
                                 const AttnWs& lay, cudaStream_t st) {
  __nv_bfloat16* p = static_cast<__nv_bfloat16*>(pk);
  return d == 64 ? launch_d<64>(B, M, r, C, dO, flags, dC, part, p, tiles_per_cta, chunks, ws, lay, st)
                 : launch_d<128>(B, M, r, C, dO, flags, dC, part, p, tiles_per_cta, chunks, ws, lay, st);
}

}  // namespace solar
