// SVD-Attention over the r factor tokens (Eq. 12) on the tensor cores (bf16 storage,
// d = 64 or 128).  One CTA per 128 candidate rows of one user:
//   TMA: candidate tile C [128 x d] and the packed per-user operands (T^T and Value_r^T,
//        each as a high and a low bf16 half) -> shared memory, 128-byte swizzle
//   tcgen05.mma: scores [128 x r] = C T (high + low half), fp32 in tensor memory
//   tcgen05.ld: one score row per thread; softmax over the r tokens entirely in that
//        thread's registers; the probabilities go back to shared memory as bf16 high/low
//   tcgen05.mma: O [128 x d] = P Value_r (hi*hi + hi*lo + lo*hi), fp32 in tensor memory
//   tcgen05.ld -> bf16 -> shared memory -> TMA store (rows past M are clipped)
// The M x r score matrix never leaves the SM.  Shared and tensor memory are reused along the
// way -- the candidate tile's buffer holds the probabilities once the scores are formed and
// the output tile after that; the output accumulator takes the scores' columns -- so that five
// CTAs (d = 64, r <= 32) share an SM and keep enough bytes in flight for the HBM.  Every wait is bounded; if one runs out the
// tile's output rows are written as NaN.
#include "sm100_ptx.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kRows = 128;                 // candidate rows per CTA = accumulator lanes
constexpr int kBoxBytes = kRows * 128;     // one 64-column box of a 128-row tile
constexpr int kErrLoad = 0x21, kErrScores = 0x22, kErrOut = 0x23;

template <int D> struct AttnCfg {
  static constexpr int KB = D / 64;                               // 64-wide K boxes of the score GEMM
  static constexpr int C_BYTES = KB * kBoxBytes;                  // candidate tile, reused for the output tile
  // T^T hi/lo: [2][KB][np rows][128 B], np = 16 * ceil(r / 16) token rows (known at launch)
  __host__ __device__ static constexpr int t_bytes(int np) { return 2 * KB * np * 128; }
  static constexpr int V_BYTES = 2 * D * 128;                     // Value_r^T hi/lo: [2][D rows][128 B]
  // Probabilities hi/lo: [2][128 rows][128 B], or [2][128 rows][64 B] (64-byte swizzle) when
  // np <= 32.  They lie over the candidate tile when they fit there (always but d = 64, np > 32).
  __host__ __device__ static constexpr bool p_narrow(int np) { return np <= 32; }
  __host__ __device__ static constexpr int p_bytes(int np) { return p_narrow(np) ? kBoxBytes : 2 * kBoxBytes; }
  __host__ __device__ static constexpr bool p_over_c(int np) { return p_bytes(np) <= C_BYTES; }
  static constexpr size_t smem(int np) {
    return (size_t)C_BYTES + t_bytes(np) + V_BYTES + (p_over_c(np) ? 0 : p_bytes(np)) + 1024;
  }
  static constexpr int TMEM_COLS = D;                             // scores (<= 64 columns), then the output (D)
};

template <int D>
__global__ void __launch_bounds__(128)
attn_umma_kernel(const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmO,
                 const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmV,
                 int r, unsigned flags, __nv_bfloat16* __restrict__ O, int M, int early_c) {
  using Cfg = AttnCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sC = base;                         // [KB][128 rows][128 B]
  uint8_t* sT = sC + Cfg::C_BYTES;            // [2][KB][np rows][128 B]
  __shared__ __align__(8) uint64_t bar_load, bar_s, bar_o;
  __shared__ uint32_t s_tmem;
  __shared__ int s_err;

  const int b = blockIdx.y, m0 = blockIdx.x * kRows;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int np = (r + 15) & ~15;              // token slots the GEMMs run over (multiple of 16)
  const int t_tile = np * 128;                // bytes of one [np rows][128 B] tile of T^T
  uint8_t* sV = sT + Cfg::t_bytes(np);        // [2][D rows][128 B]   (a multiple of 2 KB further on)
  const bool p64 = Cfg::p_narrow(np);         // probabilities in 64-byte rows
  uint8_t* sP = Cfg::p_over_c(np) ? sC : sV + Cfg::V_BYTES;   // [2][128 rows][128 or 64 B]
  const int p_half = p64 ? kBoxBytes / 2 : kBoxBytes;          // bytes of one of the two halves

  if (tid == 0) {
    s_err = 0;
    ptx::mbar_init(&bar_load, 1); ptx::mbar_init(&bar_s, 1); ptx::mbar_init(&bar_o, 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmC); ptx::prefetch_tensormap(&tmT);
    ptx::prefetch_tensormap(&tmV); ptx::prefetch_tensormap(&tmO);
  }
  if (warp == 1) ptx::tmem_alloc(&s_tmem, Cfg::TMEM_COLS);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_s = s_tmem, tmem_o = s_tmem;   // the output takes the scores' columns once they are read
  volatile int* err = &s_err;

  if (tid == 0) {
    ptx::mbar_arrive_expect_tx(&bar_load, Cfg::C_BYTES + Cfg::t_bytes(np) + Cfg::V_BYTES);
    // The packed operands come from the kernel before this one.  The candidate tile is the
    // caller's: it may be fetched ahead of the wait only when an earlier kernel of the same
    // library call has already waited for whatever ran before the call (early_c).
    if (!early_c) pdl_wait();
#pragma unroll
    for (int x = 0; x < Cfg::KB; ++x) ptx::tma_load_3d(sC + x * kBoxBytes, &tmC, &bar_load, x * 64, m0, b);
    if (early_c) pdl_wait();
#pragma unroll
    for (int x = 0; x < Cfg::KB; ++x) {
#pragma unroll
      for (int h = 0; h < 2; ++h)     // rows h*64 .. h*64+63 of the packed T^T (hi, then lo)
        ptx::tma_load_3d(sT + (h * Cfg::KB + x) * t_tile, &tmT, &bar_load, x * 64,
                         h * kTokenSlots, b);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h)
      ptx::tma_load_3d(sV + h * (D * 128), &tmV, &bar_load, 0, h * D, b);
  }

  if (tid == 32) {
    // ---- scores = C T_hi + C T_lo : M = 128, N = np, K = D -------------------------------
    if (ptx::mbar_wait(&bar_load, 0, err, kErrLoad)) {
      ptx::tc_fence_after_sync();
      const uint32_t idesc = ptx::umma_idesc_bf16(kRows, np, false, false);
      bool acc = false;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t a = ptx::smem_u32(sC) + (kk / 4) * kBoxBytes + (kk % 4) * 32;
          const uint32_t t = ptx::smem_u32(sT) + (h * Cfg::KB + kk / 4) * t_tile + (kk % 4) * 32;
          ptx::umma_bf16_ss(tmem_s, ptx::umma_smem_desc(a, 0, 1024), ptx::umma_smem_desc(t, 0, 1024), idesc, acc);
          acc = true;
        }
    }
    ptx::umma_commit(&bar_s);
  }
  __syncwarp();

  // ---- softmax over the r tokens, one candidate row per thread -------------------------
  const bool have_s = ptx::mbar_wait(&bar_s, 0, err, kErrScores);
  pdl_trigger();       // loads and the score GEMM are done: the next kernel may start launching
  __syncwarp();
  ptx::tc_fence_after_sync();
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  float p[kTokenSlots];
  {
    uint32_t v[32];
    ptx::tmem_ld_32x32(tmem_s + lane_base, v);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 32; ++i) p[i] = __uint_as_float(v[i]);
    if (np > 32) {
      ptx::tmem_ld_32x32(tmem_s + lane_base + 32, v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) p[32 + i] = __uint_as_float(v[i]);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) p[32 + i] = 0.f;
    }
  }
  if (!(flags & SOLAR_FLAG_NO_SOFTMAX)) {
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
  } else {
#pragma unroll
    for (int i = 0; i < kTokenSlots; ++i) p[i] = (i < r) ? p[i] : 0.f;
  }
  // probabilities as the A operand of the second GEMM: row tid, K = token, hi and lo halves
#pragma unroll
  for (int c = 0; c < kTokenSlots / 8; ++c) {
    if (c * 8 < np) {
      uint32_t hi[4], lo[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float x0 = p[8 * c + 2 * q], x1 = p[8 * c + 2 * q + 1];
        const float h0 = __bfloat162float(__float2bfloat16_rn(x0));
        const float h1 = __bfloat162float(__float2bfloat16_rn(x1));
        hi[q] = ptx::pack_bf16(h0, h1);
        lo[q] = ptx::pack_bf16(x0 - h0, x1 - h1);
      }
      const uint32_t off = p64 ? ptx::swz64(tid, c) : ptx::swz128(tid, c);
      *reinterpret_cast<uint4*>(sP + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
      *reinterpret_cast<uint4*>(sP + p_half + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    }
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before_sync();
  __syncthreads();

  if (tid == 32) {
    // ---- O = P_hi V_hi + P_hi V_lo + P_lo V_hi : M = 128, N = D, K = np -----------------
    ptx::tc_fence_after_sync();
    if (have_s && *err == 0) {
      const uint32_t idesc = ptx::umma_idesc_bf16(kRows, D, false, false);
      bool acc = false;
#pragma unroll
      for (int term = 0; term < 3; ++term) {
        const uint32_t pa = ptx::smem_u32(sP) + (term == 2 ? p_half : 0);
        const uint32_t vb = ptx::smem_u32(sV) + (term == 1 ? D * 128 : 0);
        for (int kk = 0; kk < np / 16; ++kk) {
          const uint64_t ad = p64 ? ptx::umma_smem_desc_sw(pa + kk * 32, 0, 512, 4)     // 64-byte rows
                                  : ptx::umma_smem_desc(pa + kk * 32, 0, 1024);
          ptx::umma_bf16_ss(tmem_o, ad, ptx::umma_smem_desc(vb + kk * 32, 0, 1024), idesc, acc);
          acc = true;
        }
      }
    }
    ptx::umma_commit(&bar_o);
  }
  __syncwarp();

  // ---- output tile: tensor memory -> bf16 -> shared memory (over the candidate tile) -----
  ptx::mbar_wait(&bar_o, 0, err, kErrOut);
  __syncwarp();
  ptx::tc_fence_after_sync();
#pragma unroll
  for (int c0 = 0; c0 < D; c0 += 32) {
    uint32_t v[32];
    ptx::tmem_ld_32x32(tmem_o + lane_base + c0, v);
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
      for (int x = 0; x < Cfg::KB; ++x) ptx::tma_store_3d(&tmO, sC + x * kBoxBytes, x * 64, m0, b);
      ptx::tma_store_commit();
      ptx::tma_store_wait_read();
    }
  } else if (m0 + tid < M) {
    // a bounded wait ran out: the rows of this tile are marked NaN instead of left stale
    uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * M + m0 + tid) * D);
    const uint4 qnan = make_uint4(0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u);
#pragma unroll
    for (int c = 0; c < D / 8; ++c) dst[c] = qnan;
  }
  if (warp == 1) ptx::tmem_dealloc(s_tmem, Cfg::TMEM_COLS);
}

template <int D>
cudaError_t launch_d(int B, int M, int r, const void* C, unsigned flags, void* O, const char* ws,
                     const AttnWs& lay, bool early_c, cudaStream_t st) {
  using Cfg = AttnCfg<D>;
  CUtensorMap tmC, tmO, tmT, tmV;
  const uint64_t pu = lay.per_user;
  bool ok = encode_tmap_bf16_3d(&tmC, C, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmO, O, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  const int np = (r + 15) & ~15;
  ok = ok && encode_tmap_bf16_3d(&tmT, ws + lay.tpk_off, D, 2 * kTokenSlots, (uint64_t)B, (uint64_t)D * 2, pu, 64,
                                 np);
  ok = ok && encode_tmap_bf16_3d(&tmV, ws + lay.vpk_off, kTokenSlots, 2 * D, (uint64_t)B, kTokenSlots * 2, pu,
                                 kTokenSlots, D);
  if (!ok) return cudaErrorInvalidValue;
  static bool limits_set[kMaxDevicesCached] = {};
  const cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&attn_umma_kernel<D>), Cfg::smem(kTokenSlots),
                                          limits_set);
  if (e != cudaSuccess) return e;
  const dim3 grid((M + kRows - 1) / kRows, B), block(128);
  return launch_pdl(attn_umma_kernel<D>, grid, block, Cfg::smem(np), st, tmC, tmO, tmT, tmV, r, flags,
                    static_cast<__nv_bfloat16*>(O), M, early_c ? 1 : 0);
}

}  // namespace

bool attn_umma_supported(int d, solar_dtype_t dt) { return dt == SOLAR_BF16 && (d == 64 || d == 128); }

cudaError_t launch_attn_umma(int B, int M, int d, int r, const void* C, unsigned flags, void* O,
                             const char* ws, const AttnWs& lay, bool early_c, cudaStream_t st) {
  if (slice_limit() > 0 && attn_pipe_supported(M, d, r, SOLAR_BF16))
    return launch_attn_pipe(B, M, r, C, flags, O, ws, lay, early_c, st);
  return d == 64 ? launch_d<64>(B, M, r, C, flags, O, ws, lay, early_c, st)
                 : launch_d<128>(B, M, r, C, flags, O, ws, lay, early_c, st);
}

}  // namespace solar
