// SVD-Attention over the factor tokens (Eq. 12), throughput form: the same arithmetic as
// attn_umma.cu -- scores C T in tensor memory, softmax over the r tokens in registers, P Value_r
// on the tensor cores, bf16 output by TMA -- but a CTA walks through MANY 128-candidate tiles of
// its user with the stages overlapped instead of taking one tile and leaving:
//   warp 4 (one thread)  streams candidate tiles through a two-stage ring with TMA;
//   warp 5 (one thread)  issues the GEMMs: the scores of tile i+1 go into the second score buffer
//                        while the other warps are still busy with tile i;
//   warps 0-3            one candidate row per thread: scores -> softmax -> P (shared memory) ->
//                        output row -> staging buffer -> TMA store.
// The per-user operands, the tensor memory and the barriers are set up once per CTA, and the
// candidate stream is kept busy from inside the CTA rather than by the CTAs that happen to share
// the SM.  Used when the process asks for throughput (solar_set_slice_limit > 0) on bf16, d = 64,
// r <= 32; a single call is better served by one tile per CTA (attn_umma.cu).
// Every wait is bounded; if one runs out the CTA's output rows are written as NaN.
#include "sm100_ptx.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kRows = 128;                 // candidate rows per tile = accumulator lanes
constexpr int kBox = kRows * 128;          // one 64-column box of a 128-row tile: 16 KB
constexpr int kD = 64;
constexpr int kStages = 2;                 // candidate-tile ring
constexpr int kTilesPerCta = 16;           // long CTAs: 2 / 4 / 8 / 16 tiles gave 8.7 / 8.1 / 7.9 / 7.6 us per step on the 16 x 2048-candidate serving shape
constexpr int kErrOps = 0x41, kErrC = 0x42, kErrS = 0x43, kErrP = 0x44, kErrO = 0x45, kErrFree = 0x46;

struct PipeCfg {
  __host__ __device__ static constexpr int t_bytes(int np) { return 2 * np * 128; }   // T^T hi/lo: [2][np rows][128 B]
  static constexpr int V_BYTES = 2 * kD * 128;      // Value_r^T hi/lo: [2][d rows][128 B]
  static constexpr int P_BYTES = kBox;              // probabilities hi/lo: [2][128 rows][64 B] (64-byte swizzle)
  static constexpr int O_BYTES = kBox;              // output staging tile
  __host__ __device__ static constexpr size_t smem(int np) {
    return (size_t)t_bytes(np) + V_BYTES + kStages * kBox + P_BYTES + O_BYTES + 1024;
  }
  static constexpr int COL_S = 0, COL_O = 64;       // two score buffers of 32 columns, then the output
  static constexpr int TMEM_COLS = 128;
};

// Barrier among the 128 row threads (warps 0-3), and the same with an OR over a predicate: every
// row thread reaches both in every iteration, so a lost wait ends the loop for all of them together.
__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ bool bar_consumers_or(bool pred) {
  uint32_t out;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.u32 q, %1, 0;\n"
      "bar.red.or.pred p, 1, 128, q;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(out) : "r"((uint32_t)pred) : "memory");
  return out != 0;
}

__global__ void __launch_bounds__(192, 1)
attn_pipe_kernel(const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmO,
                 const __grid_constant__ CUtensorMap tmT, const __grid_constant__ CUtensorMap tmV,
                 int r, unsigned flags, __nv_bfloat16* __restrict__ O, int M, int early_c, int tiles) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int np = (r + 15) & ~15;              // token slots the GEMMs run over: 16 or 32
  uint8_t* sC = base;                                   // [kStages][128 rows][128 B]
  uint8_t* sP = sC + kStages * kBox;                    // [2][128 rows][64 B]
  uint8_t* sO = sP + PipeCfg::P_BYTES;                  // [128 rows][128 B]
  uint8_t* sV = sO + PipeCfg::O_BYTES;                  // [2][64 rows][128 B]
  uint8_t* sT = sV + PipeCfg::V_BYTES;                  // [2][np rows][128 B]
  __shared__ __align__(8) uint64_t ops_bar, full_c[kStages], empty_c[kStages], s_ready[2], s_free[2], p_ready, o_ready;
  __shared__ uint32_t s_tmem;
  __shared__ int s_err;

  const int b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_my = (tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // tiles blockIdx.x, + gridDim.x, ...
  const int t_tile = np * 128;

  if (tid == 0) {
    s_err = 0;
    ptx::mbar_init(&ops_bar, 1); ptx::mbar_init(&p_ready, 4); ptx::mbar_init(&o_ready, 1);
    for (int i = 0; i < kStages; ++i) { ptx::mbar_init(&full_c[i], 1); ptx::mbar_init(&empty_c[i], 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&s_ready[i], 1); ptx::mbar_init(&s_free[i], 4); }
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmC); ptx::prefetch_tensormap(&tmT);
    ptx::prefetch_tensormap(&tmV); ptx::prefetch_tensormap(&tmO);
  }
  if (warp == 5) ptx::tmem_alloc(&s_tmem, PipeCfg::TMEM_COLS);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = s_tmem;
  volatile int* err = &s_err;

  if (warp == 4) {
    if (lane == 0) {
      // ---- producer ------------------------------------------------------------------------
      ptx::mbar_arrive_expect_tx(&ops_bar, PipeCfg::t_bytes(np) + PipeCfg::V_BYTES);
      ptx::mbar_arrive_expect_tx(&full_c[0], kBox);
      // The packed operands come from the kernel before this one.  The candidates are the
      // caller's: they may be fetched ahead of the wait only when an earlier kernel of the same
      // library call has already waited for whatever ran before the call (early_c).
      if (!early_c) pdl_wait();
      ptx::tma_load_3d(sC, &tmC, &full_c[0], 0, (int)blockIdx.x * kRows, b);
      if (early_c) pdl_wait();
#pragma unroll
      for (int h = 0; h < 2; ++h) ptx::tma_load_3d(sT + h * t_tile, &tmT, &ops_bar, 0, h * kTokenSlots, b);
#pragma unroll
      for (int h = 0; h < 2; ++h) ptx::tma_load_3d(sV + h * (kD * 128), &tmV, &ops_bar, 0, h * kD, b);
      int issued = 1;
      for (int i = 1; i < n_my; ++i) {
        const int st = i % kStages;
        if (i >= kStages && !ptx::mbar_wait(&empty_c[st], ((i / kStages) - 1) & 1, err, kErrFree)) break;
        ptx::mbar_arrive_expect_tx(&full_c[st], kBox);
        ptx::tma_load_3d(sC + st * kBox, &tmC, &full_c[st], 0, ((int)blockIdx.x + i * (int)gridDim.x) * kRows, b);
        issued = i + 1;
      }
      if (*err != 0) {
        // a wait ran out somewhere: let the copies still in flight land before the CTA leaves
        int dummy = 0;
        ptx::mbar_wait(&ops_bar, 0, &dummy, 0);
        for (int i = max(0, issued - kStages); i < issued; ++i) {
          dummy = 0;
          ptx::mbar_wait(&full_c[i % kStages], (i / kStages) & 1, &dummy, 0);
        }
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      // ---- GEMM issuer -----------------------------------------------------------------------
      const uint32_t idesc_s = ptx::umma_idesc_bf16(kRows, np, false, false);
      const uint32_t idesc_o = ptx::umma_idesc_bf16(kRows, kD, false, false);
      bool ok = ptx::mbar_wait(&ops_bar, 0, err, kErrOps);
      // scores of tile i = C T_hi + C T_lo : M = 128, N = np, K = 64, into score buffer i & 1
      auto scores = [&](int i) {
        const int st = i % kStages, sb = i & 1;
        if (!ptx::mbar_wait(&full_c[st], (i / kStages) & 1, err, kErrC)) return false;
        if (i >= 2 && !ptx::mbar_wait(&s_free[sb], ((i >> 1) - 1) & 1, err, kErrFree)) return false;
        ptx::tc_fence_after_sync();
        const uint32_t a0 = ptx::smem_u32(sC + st * kBox), t0 = ptx::smem_u32(sT);
        bool acc = false;
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            ptx::umma_bf16_ss(tmem + PipeCfg::COL_S + 32 * sb, ptx::umma_smem_desc(a0 + kk * 32, 0, 1024),
                              ptx::umma_smem_desc(t0 + h * t_tile + kk * 32, 0, 1024), idesc_s, acc);
            acc = true;
          }
        ptx::umma_commit(&s_ready[sb]);     // the scores are there ...
        ptx::umma_commit(&empty_c[st]);     // ... and the candidate stage has been read
        return true;
      };
      ok = ok && scores(0);
      for (int i = 0; i < n_my && ok; ++i) {
        if (i + 1 < n_my) ok = scores(i + 1);
        if (!ok) break;
        // O = P_hi V_hi + P_hi V_lo + P_lo V_hi : M = 128, N = 64, K = np
        if (!ptx::mbar_wait(&p_ready, i & 1, err, kErrP)) { ok = false; break; }
        ptx::tc_fence_after_sync();
        bool acc = false;
#pragma unroll
        for (int term = 0; term < 3; ++term) {
          const uint32_t pa = ptx::smem_u32(sP) + (term == 2 ? kBox / 2 : 0);
          const uint32_t vb = ptx::smem_u32(sV) + (term == 1 ? kD * 128 : 0);
          for (int kk = 0; kk < np / 16; ++kk) {
            ptx::umma_bf16_ss(tmem + PipeCfg::COL_O, ptx::umma_smem_desc_sw(pa + kk * 32, 0, 512, 4),
                              ptx::umma_smem_desc(vb + kk * 32, 0, 1024), idesc_o, acc);
            acc = true;
          }
        }
        ptx::umma_commit(&o_ready);
      }
    }
  } else {
    // ---- one candidate row per thread ----------------------------------------------------------
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    for (int i = 0; i < n_my; ++i) {
      const int sb = i & 1;
      const int m0 = ((int)blockIdx.x + i * (int)gridDim.x) * kRows;
      const bool have_s = ptx::mbar_wait(&s_ready[sb], (i >> 1) & 1, err, kErrS);
      ptx::tc_fence_after_sync();
      float p[32];
      {
        uint32_t v[32];
        ptx::tmem_ld_32x32(tmem + PipeCfg::COL_S + 32 * sb + lane_base, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) p[j] = __uint_as_float(v[j]);
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0 && have_s) ptx::mbar_arrive(&s_free[sb]);      // the score buffer may take tile i + 2
      if (!(flags & SOLAR_FLAG_NO_SOFTMAX)) {
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < 32; ++j) mx = (j < r) ? fmaxf(mx, p[j]) : mx;
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          p[j] = (j < r) ? ptx::fast_exp2((p[j] - mx) * 1.4426950408889634f) : 0.f;
          sum += p[j];
        }
        const float inv = 1.f / sum;
#pragma unroll
        for (int j = 0; j < 32; ++j) p[j] *= inv;
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) p[j] = (j < r) ? p[j] : 0.f;
      }
      // probabilities as the A operand of the second GEMM: row tid, K = token, hi and lo halves
#pragma unroll
      for (int c = 0; c < 4; ++c) {
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
          const uint32_t off = ptx::swz64(tid, c);
          *reinterpret_cast<uint4*>(sP + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
          *reinterpret_cast<uint4*>(sP + kBox / 2 + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
      }
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0 && have_s) ptx::mbar_arrive(&p_ready);
      // the output tile: tensor memory -> bf16 -> staging buffer -> TMA store
      const bool have_o = have_s && ptx::mbar_wait(&o_ready, i & 1, err, kErrO);
      ptx::tc_fence_after_sync();
      if (tid == 0 && i > 0) ptx::tma_store_wait_read();   // the previous tile has left the staging buffer
      if (bar_consumers_or(!have_o)) break;                // uniform: nobody is left behind at a barrier
#pragma unroll
      for (int c0 = 0; c0 < kD; c0 += 32) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(tmem + PipeCfg::COL_O + lane_base + c0, v);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint4 w = make_uint4(
              ptx::pack_bf16(__uint_as_float(v[8 * c + 0]), __uint_as_float(v[8 * c + 1])),
              ptx::pack_bf16(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3])),
              ptx::pack_bf16(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5])),
              ptx::pack_bf16(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7])));
          *reinterpret_cast<uint4*>(sO + ptx::swz128(tid, c0 / 8 + c)) = w;
        }
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before_sync();
      bar_consumers();
      if (tid == 0) {
        ptx::tma_store_3d(&tmO, sO, 0, m0, b);
        ptx::tma_store_commit();
      }
    }
    if (tid == 0) ptx::tma_store_wait_read();
  }
  __syncwarp();
  pdl_trigger();       // by every thread: the next kernel starts launching when the last CTA is this far
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (s_err != 0 && tid < kRows) {
    // a bounded wait ran out: every row of this CTA's tiles is marked NaN instead of left stale
    const uint4 qnan = make_uint4(0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u, 0x7fc07fc0u);
    for (int i = 0; i < n_my; ++i) {
      const int row = ((int)blockIdx.x + i * (int)gridDim.x) * kRows + tid;
      if (row < M) {
        uint4* dst = reinterpret_cast<uint4*>(O + ((size_t)b * M + row) * kD);
#pragma unroll
        for (int c = 0; c < kD / 8; ++c) dst[c] = qnan;
      }
    }
  }
  if (warp == 5) ptx::tmem_dealloc(tmem, PipeCfg::TMEM_COLS);
}

}  // namespace

bool attn_pipe_supported(int M, int d, int r, solar_dtype_t dt) {
  return dt == SOLAR_BF16 && d == kD && r <= 32 && (M + kRows - 1) / kRows >= 4;
}

cudaError_t launch_attn_pipe(int B, int M, int r, const void* C, unsigned flags, void* O, const char* ws,
                             const AttnWs& lay, bool early_c, cudaStream_t st) {
  CUtensorMap tmC, tmO, tmT, tmV;
  const uint64_t pu = lay.per_user;
  const int np = (r + 15) & ~15;
  bool ok = encode_tmap_bf16_3d(&tmC, C, kD, (uint64_t)M, (uint64_t)B, (uint64_t)kD * 2, (uint64_t)M * kD * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmO, O, kD, (uint64_t)M, (uint64_t)B, (uint64_t)kD * 2, (uint64_t)M * kD * 2, 64, kRows);
  ok = ok && encode_tmap_bf16_3d(&tmT, ws + lay.tpk_off, kD, 2 * kTokenSlots, (uint64_t)B, (uint64_t)kD * 2, pu, 64, np);
  ok = ok && encode_tmap_bf16_3d(&tmV, ws + lay.vpk_off, kTokenSlots, 2 * kD, (uint64_t)B, kTokenSlots * 2, pu,
                                 kTokenSlots, kD);
  if (!ok) return cudaErrorInvalidValue;
  static bool limits_set[kMaxDevicesCached] = {};
  const cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&attn_pipe_kernel), PipeCfg::smem(32), limits_set);
  if (e != cudaSuccess) return e;
  const int tiles = (M + kRows - 1) / kRows;
  const int per_user = (tiles + kTilesPerCta - 1) / kTilesPerCta;
  return launch_pdl(attn_pipe_kernel, dim3(per_user, B), dim3(192), PipeCfg::smem(np), st, tmC, tmO, tmT, tmV, r, flags,
                    static_cast<__nv_bfloat16*>(O), M, early_c ? 1 : 0, tiles);
}

}  // namespace solar
