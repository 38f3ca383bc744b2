// Softmax attention over the N history positions evaluated through the rank-r factors
// (bf16 storage, d = 64 or 128, r = 16, 32 or 64):
//   O = softmax_N( scale * (C W_Q W_K^T V) (U Sigma)^T ) (U Sigma) (V^T W_V)
// On a history of rank <= r this IS the softmax attention of Eq. 6-7 (H = U Sigma V^T makes
// Key = U Sigma V^T W_K and Value = U Sigma V^T W_V), at O(N M r) instead of O(N M d); it
// is not the paper's SVD-Attention operator, which removes U (Eq. 10) and takes the softmax
// over the r factor tokens.
//
// One CTA per 128 candidates of one user, flash-attention style, everything on chip:
//   Q' [128 x r] = C A1 (A1 = scale log2(e) W_Q W_K^T V, hi + lo bf16 halves), tcgen05.mma
//   for each tile of 128 positions (TMA, two stages):
//     S [128 x 128] = Q' US_tile^T          tcgen05.mma, US tile as a K-major operand
//     one score row per thread: running max, exp2, running sum -- registers only
//     Y_tile [128 x r] = P US_tile          tcgen05.mma, the SAME tile as an MN-major operand
//     y = y * 2^(m_old - m_new) + Y_tile    (the accumulator lives in registers)
//   O [128 x d] = (y / l) B1  (B1 = V^T W_V, hi/lo halves), tcgen05.mma, TMA store.
// The N x M score matrix never exists outside tensor memory.  Every wait is bounded; if one
// runs out the tile's output rows are written as NaN.
#include "sm100_ptx.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kRows = 128;                 // candidates per CTA = accumulator lanes
constexpr int kPos = 128;                  // history positions per tile
constexpr int kBox = kRows * 128;          // bytes of a [128 rows][128 B] swizzled box
constexpr int kErrLoad = 0x31, kErrQ = 0x32, kErrTile = 0x33, kErrS = 0x34, kErrY = 0x35, kErrO = 0x36;

template <int D, int R> struct FlashCfg {
  static constexpr int KB = D / 64;                   // 64-wide K boxes of C
  static constexpr int RB = R * 2;                    // bytes of one US row = swizzle span of its tile
  static constexpr uint32_t US_LAYOUT = (R == 64) ? 2u : (R == 32) ? 4u : 6u;   // descriptor swizzle code
  static constexpr int C_BYTES = KB * kBox;           // candidate tile; later the output tile
  static constexpr int T_BYTES = 2 * KB * R * 128;    // A1^T hi/lo: [2][KB][R rows][128 B]
  static constexpr int V_BYTES = 2 * D * 128;         // B1^T hi/lo: [2][D rows][128 B] (K = token)
  static constexpr int Q_BYTES = 2 * kBox;            // Q' hi/lo, later y hi/lo: [2][128][128 B]
  static constexpr int P_BYTES = 2 * kBox;            // probabilities: [2 boxes of 64 positions][128][128 B]
  static constexpr int US_TILE = kPos * RB;           // one tile of U Sigma
  // the candidate tile (read once, by the Q' GEMM) and the output tile (written last) share
  // the probabilities' buffer
  static_assert(C_BYTES <= P_BYTES, "C and O tiles live in the P buffer");
  static constexpr size_t SMEM = (size_t)T_BYTES + V_BYTES + Q_BYTES + P_BYTES + 2 * US_TILE + 1024;
  static constexpr int COL_Q = 0, COL_S = 64, COL_O = 192;      // tensor-memory columns
  static constexpr int TMEM_COLS = (D == 64) ? 256 : 512;
};

// Writes R fp32 values of this thread's row as bf16 high and low halves into two swizzled
// K-major tiles (hi at `dst`, lo one box further).
template <int R>
__device__ __forceinline__ void store_hi_lo(uint8_t* dst, int row, const float (&x)[R]) {
#pragma unroll
  for (int c = 0; c < R / 8; ++c) {
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float a = x[8 * c + 2 * q], b = x[8 * c + 2 * q + 1];
      const float ha = __bfloat162float(__float2bfloat16_rn(a)), hb = __bfloat162float(__float2bfloat16_rn(b));
      hi[q] = ptx::pack_bf16(ha, hb);
      lo[q] = ptx::pack_bf16(a - ha, b - hb);
    }
    *reinterpret_cast<uint4*>(dst + ptx::swz128(row, c)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(dst + kBox + ptx::swz128(row, c)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

// Loads this thread's row of a tensor-memory block of R (<= 64) fp32 columns.
template <int R>
__device__ __forceinline__ void tmem_row(uint32_t taddr, float (&x)[R]) {
  uint32_t v[32];
  ptx::tmem_ld_32x32(taddr, v);
  ptx::tmem_ld_wait();
#pragma unroll
  for (int i = 0; i < (R < 32 ? R : 32); ++i) x[i] = __uint_as_float(v[i]);
  if constexpr (R > 32) {
    ptx::tmem_ld_32x32(taddr + 32, v);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < R - 32; ++i) x[32 + i] = __uint_as_float(v[i]);
  }
}

template <int D, int R>
__global__ void __launch_bounds__(128, 2)
flash_factored_kernel(const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmO,
                      const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmV,
                      const __grid_constant__ CUtensorMap tmUS, int N, int M, __nv_bfloat16* __restrict__ O) {
  using Cfg = FlashCfg<D, R>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sT = base;                         // [2][KB][R][128 B]
  uint8_t* sV = sT + Cfg::T_BYTES;            // [2][D][128 B]
  uint8_t* sQ = sV + Cfg::V_BYTES;            // [2][128][128 B]
  uint8_t* sP = sQ + Cfg::Q_BYTES;            // [2][128][128 B]
  uint8_t* sC = sP;                           // [KB][128][128 B]  candidate tile first, output tile last
  uint8_t* sUS = sP + Cfg::P_BYTES;           // [2 stages][128][RB]
  __shared__ __align__(8) uint64_t bar_load, bar_q, bar_s, bar_y, bar_o, bar_us[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_err;

  const int b = blockIdx.y, m0 = blockIdx.x * kRows;
  const int tid = threadIdx.x, warp = tid >> 5;
  const int ntiles = (N + kPos - 1) / kPos;

  if (tid == 0) {
    s_err = 0;
    ptx::mbar_init(&bar_load, 1); ptx::mbar_init(&bar_q, 1); ptx::mbar_init(&bar_s, 1);
    ptx::mbar_init(&bar_y, 1); ptx::mbar_init(&bar_o, 1);
    ptx::mbar_init(&bar_us[0], 1); ptx::mbar_init(&bar_us[1], 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmC); ptx::prefetch_tensormap(&tmT); ptx::prefetch_tensormap(&tmV);
    ptx::prefetch_tensormap(&tmUS); ptx::prefetch_tensormap(&tmO);
  }
  if (warp == 1) ptx::tmem_alloc(&s_tmem, Cfg::TMEM_COLS);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  const uint32_t tm_q = s_tmem + Cfg::COL_Q, tm_s = s_tmem + Cfg::COL_S, tm_o = s_tmem + Cfg::COL_O;
  volatile int* err = &s_err;

  if (tid == 0) {
    ptx::mbar_arrive_expect_tx(&bar_load, Cfg::C_BYTES + Cfg::T_BYTES + Cfg::V_BYTES);
#pragma unroll
    for (int x = 0; x < Cfg::KB; ++x) ptx::tma_load_3d(sC + x * kBox, &tmC, &bar_load, x * 64, m0, b);
    pdl_wait();        // the packed operands and U Sigma come from earlier kernels on the stream
#pragma unroll
    for (int x = 0; x < Cfg::KB; ++x)
#pragma unroll
      for (int h = 0; h < 2; ++h)
        ptx::tma_load_3d(sT + (h * Cfg::KB + x) * (R * 128), &tmT, &bar_load, x * 64, h * kTokenSlots, b);
#pragma unroll
    for (int h = 0; h < 2; ++h) ptx::tma_load_3d(sV + h * (D * 128), &tmV, &bar_load, 0, h * D, b);
    for (int t = 0; t < 2 && t < ntiles; ++t) {
      ptx::mbar_arrive_expect_tx(&bar_us[t], Cfg::US_TILE);
      ptx::tma_load_3d(sUS + t * Cfg::US_TILE, &tmUS, &bar_us[t], 0, t * kPos, b);
    }
  }

  if (tid == 32) {
    // ---- Q' = C A1_hi + C A1_lo : M = 128, N = R, K = D ------------------------------------
    if (ptx::mbar_wait(&bar_load, 0, err, kErrLoad)) {
      ptx::tc_fence_after_sync();
      const uint32_t idesc = ptx::umma_idesc_bf16(kRows, R, false, false);
      bool acc = false;
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t a = ptx::smem_u32(sC) + (kk / 4) * kBox + (kk % 4) * 32;
          const uint32_t t = ptx::smem_u32(sT) + (h * Cfg::KB + kk / 4) * (R * 128) + (kk % 4) * 32;
          ptx::umma_bf16_ss(tm_q, ptx::umma_smem_desc(a, 0, 1024), ptx::umma_smem_desc(t, 0, 1024), idesc, acc);
          acc = true;
        }
    }
    ptx::umma_commit(&bar_q);
  }
  __syncwarp();
  ptx::mbar_wait(&bar_q, 0, err, kErrQ);
  __syncwarp();
  ptx::tc_fence_after_sync();
  {
    float q[R];
    tmem_row<R>(tm_q + lane_base, q);
    store_hi_lo<R>(sQ, tid, q);
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before_sync();
  __syncthreads();

  // ---- the positions, 128 at a time ----------------------------------------------------
  float y[R];
#pragma unroll
  for (int i = 0; i < R; ++i) y[i] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;
  const uint32_t idesc_s = ptx::umma_idesc_bf16(kRows, kPos, false, false);   // S = Q' US^T
  const uint32_t idesc_y = ptx::umma_idesc_bf16(kRows, R, false, true);       // Y = P US (US MN-major)
  // (after a lost wait every thread still walks through all the tiles -- the barriers below
  // need all of them -- but the waits return at once and nothing more is issued)
  for (int t = 0; t < ntiles; ++t) {
    const int st = t & 1;
    const uint32_t us = ptx::smem_u32(sUS + st * Cfg::US_TILE);
    if (tid == 32) {
      if (ptx::mbar_wait(&bar_us[st], (t >> 1) & 1, err, kErrTile)) {
        ptx::tc_fence_after_sync();
        bool acc = false;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int kk = 0; kk < R / 16; ++kk) {
            // A: Q' half h, K-major, 128-byte rows.  B: the tile's rows are the K-major operand
            // rows (one position each, RB bytes, swizzle span RB, 8-row atoms of 8*RB bytes).
            const uint64_t a = ptx::umma_smem_desc(ptx::smem_u32(sQ) + h * kBox + kk * 32, 0, 1024);
            const uint64_t bd = ptx::umma_smem_desc_sw(us + kk * 32, 0, 8 * Cfg::RB, Cfg::US_LAYOUT);
            ptx::umma_bf16_ss(tm_s, a, bd, idesc_s, acc);
            acc = true;
          }
      }
      ptx::umma_commit(&bar_s);
    }
    __syncwarp();
    ptx::mbar_wait(&bar_s, t & 1, err, kErrS);
    __syncwarp();
    ptx::tc_fence_after_sync();

    // this thread's 128 scores (already in log2 units): running max, exp2, running sum
    float s[kPos];
    {
      // all four loads in flight, one wait
      uint32_t v0[32], v1[32], v2[32], v3[32];
      ptx::tmem_ld_32x32(tm_s + lane_base, v0);
      ptx::tmem_ld_32x32(tm_s + lane_base + 32, v1);
      ptx::tmem_ld_32x32(tm_s + lane_base + 64, v2);
      ptx::tmem_ld_32x32(tm_s + lane_base + 96, v3);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        s[i] = __uint_as_float(v0[i]);      s[32 + i] = __uint_as_float(v1[i]);
        s[64 + i] = __uint_as_float(v2[i]); s[96 + i] = __uint_as_float(v3[i]);
      }
    }
    const int valid = N - t * kPos;                 // positions past N hold zero-filled rows
    if (valid < kPos) {
#pragma unroll
      for (int j = 0; j < kPos; ++j) s[j] = (j < valid) ? s[j] : -INFINITY;
    }
    // eight independent chains for the maximum and for the sum: with two warps per scheduler a
    // 128-long dependent chain would be exposed latency
    float mx[8], sm8[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) mx[q] = s[q];
#pragma unroll
    for (int j = 8; j < kPos; ++j) mx[j & 7] = fmaxf(mx[j & 7], s[j]);
    const float m_new = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                              fmaxf(fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])), m_run));
    const float alpha = ptx::fast_exp2(m_run - m_new);         // 0 on the first tile (m_run = -inf)
#pragma unroll
    for (int q = 0; q < 8; ++q) sm8[q] = 0.f;
#pragma unroll
    for (int j = 0; j < kPos; ++j) {
      s[j] = ptx::fast_exp2(s[j] - m_new);                     // masked positions: 2^-inf = 0
      sm8[j & 7] += s[j];
    }
    const float sum = ((sm8[0] + sm8[1]) + (sm8[2] + sm8[3])) + ((sm8[4] + sm8[5]) + (sm8[6] + sm8[7]));
    l_run = fmaf(l_run, alpha, sum);
    m_run = m_new;
#pragma unroll
    for (int c = 0; c < kPos / 8; ++c) {            // P as bf16, K-major: two boxes of 64 positions
      const uint4 w = make_uint4(ptx::pack_bf16(s[8 * c], s[8 * c + 1]), ptx::pack_bf16(s[8 * c + 2], s[8 * c + 3]),
                                 ptx::pack_bf16(s[8 * c + 4], s[8 * c + 5]), ptx::pack_bf16(s[8 * c + 6], s[8 * c + 7]));
      *reinterpret_cast<uint4*>(sP + (c / 8) * kBox + ptx::swz128(tid, c % 8)) = w;
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();

    if (tid == 32) {
      ptx::tc_fence_after_sync();
      if (*err == 0) {
#pragma unroll
        for (int kk = 0; kk < kPos / 16; ++kk) {
          // A: P, K-major.  B: the same U Sigma tile read MN-major: 16 positions = two groups
          // of 8 rows (8*RB bytes apart); its R columns are one MN block.
          const uint64_t a = ptx::umma_smem_desc(ptx::smem_u32(sP) + (kk / 4) * kBox + (kk % 4) * 32, 0, 1024);
          const uint64_t bd = ptx::umma_smem_desc_sw(us + kk * 16 * Cfg::RB, 0, 8 * Cfg::RB, Cfg::US_LAYOUT);
          ptx::umma_bf16_ss(tm_q, a, bd, idesc_y, kk != 0);
        }
      }
      ptx::umma_commit(&bar_y);
    }
    __syncwarp();
    ptx::mbar_wait(&bar_y, t & 1, err, kErrY);
    __syncwarp();
    ptx::tc_fence_after_sync();
    if (tid == 0 && t + 2 < ntiles && *err == 0) {  // this stage's tile has been consumed: refill it
      ptx::mbar_arrive_expect_tx(&bar_us[st], Cfg::US_TILE);
      ptx::tma_load_3d(sUS + st * Cfg::US_TILE, &tmUS, &bar_us[st], 0, (t + 2) * kPos, b);
    }
    {
      float yt[R];
      tmem_row<R>(tm_q + lane_base, yt);
#pragma unroll
      for (int i = 0; i < R; ++i) y[i] = fmaf(y[i], alpha, yt[i]);
    }
    ptx::tc_fence_before_sync();
  }
  pdl_trigger();

  // ---- O = (y / l) B1 : M = 128, N = D, K = R, hi*hi + hi*lo + lo*hi ---------------------
  {
    const float inv = 1.f / l_run;
#pragma unroll
    for (int i = 0; i < R; ++i) y[i] *= inv;
    store_hi_lo<R>(sQ, tid, y);
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (tid == 32) {
    ptx::tc_fence_after_sync();
    if (*err == 0) {
      const uint32_t idesc = ptx::umma_idesc_bf16(kRows, D, false, false);
      bool acc = false;
#pragma unroll
      for (int term = 0; term < 3; ++term) {
        const uint32_t ya = ptx::smem_u32(sQ) + (term == 2 ? kBox : 0);
        const uint32_t vb = ptx::smem_u32(sV) + (term == 1 ? D * 128 : 0);
#pragma unroll
        for (int kk = 0; kk < R / 16; ++kk) {
          ptx::umma_bf16_ss(tm_o, ptx::umma_smem_desc(ya + kk * 32, 0, 1024),
                            ptx::umma_smem_desc(vb + kk * 32, 0, 1024), idesc, acc);
          acc = true;
        }
      }
    }
    ptx::umma_commit(&bar_o);
  }
  __syncwarp();
  ptx::mbar_wait(&bar_o, 0, err, kErrO);
  __syncwarp();
  ptx::tc_fence_after_sync();
#pragma unroll
  for (int c0 = 0; c0 < D; c0 += 32) {
    uint32_t v[32];
    ptx::tmem_ld_32x32(tm_o + lane_base + c0, v);
    ptx::tmem_ld_wait();
    uint8_t* box = sC + (c0 / 64) * kBox;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint4 w = make_uint4(ptx::pack_bf16(__uint_as_float(v[8 * c + 0]), __uint_as_float(v[8 * c + 1])),
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
      for (int x = 0; x < Cfg::KB; ++x) ptx::tma_store_3d(&tmO, sC + x * kBox, x * 64, m0, b);
      ptx::tma_store_commit();
      ptx::tma_store_wait_read();
    }
  } else if (m0 + tid < M) {
    uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * M + m0 + tid) * D);
    const uint4 qnan = make_uint4(0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u);
#pragma unroll
    for (int c = 0; c < D / 8; ++c) dst[c] = qnan;
  }
  if (warp == 1) ptx::tmem_dealloc(s_tmem, Cfg::TMEM_COLS);
}

template <int D, int R>
cudaError_t launch_dr(int B, int M, int N, const void* C, const void* US, void* O, const char* ws,
                      const AttnWs& lay, cudaStream_t st) {
  using Cfg = FlashCfg<D, R>;
  CUtensorMap tmC, tmO, tmT, tmV, tmUS;
  const uint64_t pu = lay.per_user;
  bool ok = encode_tmap_bf16_3d(&tmC, C, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmO, O, D, (uint64_t)M, (uint64_t)B, (uint64_t)D * 2, (uint64_t)M * D * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmT, ws + lay.tpk_off, D, 2 * kTokenSlots, (uint64_t)B, (uint64_t)D * 2, pu, 64, R);
  ok = ok && encode_tmap_bf16_3d(&tmV, ws + lay.vpk_off, kTokenSlots, 2 * D, (uint64_t)B, kTokenSlots * 2, pu,
                                 kTokenSlots, D);
  ok = ok && encode_tmap_bf16_3d_sw(&tmUS, US, R, (uint64_t)N, (uint64_t)B, (uint64_t)R * 2, (uint64_t)N * R * 2, R,
                                    kPos, Cfg::RB);
  if (!ok) return cudaErrorInvalidValue;
  static bool limits_set[kMaxDevicesCached] = {};
  const cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&flash_factored_kernel<D, R>), Cfg::SMEM,
                                          limits_set);
  if (e != cudaSuccess) return e;
  const dim3 grid((M + kRows - 1) / kRows, B), block(128);
  return launch_pdl(flash_factored_kernel<D, R>, grid, block, Cfg::SMEM, st, tmC, tmO, tmT, tmV, tmUS, N, M,
                    static_cast<__nv_bfloat16*>(O));
}

}  // namespace

bool flash_factored_supported(int d, int r, solar_dtype_t dt) {
  return dt == SOLAR_BF16 && (d == 64 || d == 128) && (r == 16 || r == 32 || r == 64);
}

cudaError_t launch_flash_factored(int B, int M, int N, int d, int r, const void* C, const void* US, void* O,
                                  const char* ws, const AttnWs& lay, cudaStream_t st) {
#define SOLAR_FF(DD, RR) \
  if (d == DD && r == RR) return launch_dr<DD, RR>(B, M, N, C, US, O, ws, lay, st);
  SOLAR_FF(64, 16) SOLAR_FF(64, 32) SOLAR_FF(64, 64) SOLAR_FF(128, 16) SOLAR_FF(128, 32) SOLAR_FF(128, 64)
#undef SOLAR_FF
  return cudaErrorInvalidValue;
}

}  // namespace solar
