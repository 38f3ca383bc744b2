// Right-multiplication of every history by a per-user matrix on the tensor cores (bf16
// storage, d = 64 or 128):   Out_b = H_b X_b,   X_b [d][q] fp32,  q <= 128.
// Two callers: the optional left factor  US = U Sigma = H V  (q = r; Eq. 10 eliminates U
// from the forward pass, this second streaming pass over H serves attention over the N
// positions through the factors) and the backward pass of the SVD, dH = H K (q = d; Eq. 15
// with U = H V Sigma^-1).
//
// One CTA per (user, row slice), the same slicing as the Gram pass.  Warp 4 streams the
// slice's 128-row tiles of H through a ring of shared-memory stages with TMA; warp 5
// issues tcgen05.mma with the tile as the K-major A operand (M = 128 rows, K = d) and
// X^T, split into a high and a low bf16 half, as the K-major B operand, into one of two
// accumulators in tensor memory; warps 0-3 read the finished accumulator (one row per
// thread), round to bf16 and store the rows, while the next tile is being multiplied
// into the other accumulator.  H is read from HBM once and never passes through registers.
#include "sm100_ptx.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kTileRows = kGramTileRows;
constexpr int kEpiThreads = 128, kProducerWarp = 4, kMmaWarp = 5, kThreads = 192;
constexpr int kMaxCols = 128;                // q <= 128 output columns
constexpr int kErrProducer = 0x41, kErrMma = 0x42, kErrEpilogue = 0x43;

template <int D> struct UsCfg {
  static constexpr int KB = D / 64;                          // 64-column TMA boxes per tile
  static constexpr int BOX_BYTES = kTileRows * 128;          // 16 KB: 128 rows x 64 bf16
  static constexpr int TILE_BYTES = KB * BOX_BYTES;
  static constexpr int STAGES = (D == 64) ? 6 : 4;
  // ring + X^T as [2 halves][KB][np rows][128 B] + slack to align to 1024
  static constexpr size_t smem(int np) { return (size_t)STAGES * TILE_BYTES + (size_t)2 * KB * np * 128 + 1024; }
};

// byte offset of 16-byte chunk c of row `row` in a [rows][128 B] tile with the 128-byte swizzle
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
project_us_umma_kernel(const __grid_constant__ CUtensorMap tmap, const float* __restrict__ V,
                       __nv_bfloat16* __restrict__ US, int N, int r, int chunk_rows) {
  // V is the per-user matrix X [D][r] and US the output [N][r]; r stands for q here.
  using Cfg = UsCfg<D>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sV = tiles + (size_t)STAGES * Cfg::TILE_BYTES;
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_free[2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_err;

  const int b = blockIdx.y, s = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = s * chunk_rows;
  const int row1 = min(N, row0 + chunk_rows);
  const int ntiles = (row1 - row0 + kTileRows - 1) / kTileRows;
  const int np = (r + 15) & ~15;              // columns the GEMM runs over (multiple of 16)
  const int v_tile = np * 128;                // bytes of one [np rows][128 B] tile of V^T
  const int acc_cols = np > 64 ? 128 : 64;    // tensor-memory columns per accumulator

  if (tid == 0) {
    s_err = 0;
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&full_bar[i], 1); ptx::mbar_init(&empty_bar[i], 1); }
    for (int i = 0; i < 2; ++i) { ptx::mbar_init(&acc_full[i], 1); ptx::mbar_init(&acc_free[i], kEpiThreads); }
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap);
  }
  if (warp == kMmaWarp) ptx::tmem_alloc(&s_tmem, 2 * acc_cols);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = s_tmem;
  volatile int* err = &s_err;

  auto load_tile = [&](int t) {
    const int st = t % STAGES;
    ptx::mbar_arrive_expect_tx(&full_bar[st], Cfg::TILE_BYTES);
#pragma unroll
    for (int x = 0; x < Cfg::KB; ++x)
      ptx::tma_load_3d(tiles + (size_t)st * Cfg::TILE_BYTES + x * Cfg::BOX_BYTES, &tmap, &full_bar[st],
                       x * 64, row0 + t * kTileRows, b);
  };
  // the first tiles are on their way while V^T is being packed
  const int primed = min(ntiles, STAGES);
  if (warp == kProducerWarp && lane == 0)
    for (int t = 0; t < primed; ++t) load_tile(t);

  // V^T as two K-major bf16 operands: row i (factor), K = k (feature); rows r .. np-1 zero
  for (int e = tid; e < np * D; e += kThreads) {
    const int k = e / np, i = e % np;
    const float v = i < r ? V[((size_t)b * D + k) * r + i] : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    const uint32_t off = (uint32_t)(k / 64) * v_tile + ptx::swz128(i, (k % 64) / 8) + (k % 8) * 2;
    *reinterpret_cast<__nv_bfloat16*>(sV + off) = hi;
    *reinterpret_cast<__nv_bfloat16*>(sV + Cfg::KB * v_tile + off) = lo;
  }
  ptx::fence_proxy_async_smem();
  __syncthreads();

  if (warp == kProducerWarp) {
    if (lane == 0) {
      int issued = primed;
      for (int t = primed; t < ntiles; ++t) {
        if (!ptx::mbar_wait(&empty_bar[t % STAGES], ((t / STAGES) - 1) & 1, err, kErrProducer)) break;
        load_tile(t);
        issued = t + 1;
      }
      if (*err != 0) {
        // a wait ran out somewhere: let the copies still in flight land before the CTA leaves
        for (int t = max(0, issued - STAGES); t < issued; ++t) {
          int dummy = 0;
          ptx::mbar_wait(&full_bar[t % STAGES], (t / STAGES) & 1, &dummy, 0);
        }
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      const uint32_t idesc = ptx::umma_idesc_bf16(kTileRows, np, false, false);
      const uint32_t vbase = ptx::smem_u32(sV);
      for (int t = 0; t < ntiles; ++t) {
        const int st = t % STAGES, a = t & 1;
        if (!ptx::mbar_wait(&full_bar[st], (t / STAGES) & 1, err, kErrMma)) break;
        if (t >= 2 && !ptx::mbar_wait(&acc_free[a], ((t >> 1) - 1) & 1, err, kErrMma)) break;
        ptx::tc_fence_after_sync();
        const uint32_t hbase = ptx::smem_u32(tiles + (size_t)st * Cfg::TILE_BYTES);
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t ha = hbase + (kk / 4) * Cfg::BOX_BYTES + (kk % 4) * 32;
            const uint32_t vb = vbase + (h * Cfg::KB + kk / 4) * v_tile + (kk % 4) * 32;
            ptx::umma_bf16_ss(tmem + a * acc_cols, ptx::umma_smem_desc(ha, 0, 1024),
                              ptx::umma_smem_desc(vb, 0, 1024), idesc, (h | kk) != 0);
          }
        ptx::umma_commit(&empty_bar[st]);     // the stage is free once these MMAs have read it
        ptx::umma_commit(&acc_full[a]);
      }
    }
  } else {
    // ---- epilogue warps: accumulator row tid -> bf16 -> US[b, n, 0:r] ------------------
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const bool vec = (r % 8) == 0 && (reinterpret_cast<uintptr_t>(US) & 15) == 0;   // rows start on 16-byte boundaries
    int t = 0;
    for (; t < ntiles; ++t) {
      const int a = t & 1;
      // the warp leaves together: the tensor-memory loads below are warp-wide
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&acc_full[a], (t >> 1) & 1, err, kErrEpilogue))) break;
      ptx::tc_fence_after_sync();
      const int n = row0 + t * kTileRows + tid;
      __nv_bfloat16* o = US + ((size_t)b * N + (n < N ? n : 0)) * r;
      for (int c0 = 0; c0 < np; c0 += 32) {
        uint32_t v[32];
        ptx::tmem_ld_32x32(tmem + lane_base + a * acc_cols + c0, v);
        ptx::tmem_ld_wait();
        if (c0 + 32 >= np) {                     // last chunk read: the accumulator may be overwritten
          ptx::tc_fence_before_sync();
          ptx::mbar_arrive(&acc_free[a]);
        }
        if (n < N) {
          if (vec) {
            uint4* o4 = reinterpret_cast<uint4*>(o + c0);
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if (c0 + 8 * c < r)
                o4[c] = make_uint4(ptx::pack_bf16(__uint_as_float(v[8 * c]), __uint_as_float(v[8 * c + 1])),
                                   ptx::pack_bf16(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3])),
                                   ptx::pack_bf16(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5])),
                                   ptx::pack_bf16(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7])));
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i < r) o[c0 + i] = __float2bfloat16_rn(__uint_as_float(v[i]));
          }
        }
      }
    }
    // a wait ran out: the rows that were not produced read as NaN
    for (; t < ntiles; ++t) {
      const int n = row0 + t * kTileRows + tid;
      if (n < N)
        for (int i = 0; i < r; ++i) US[((size_t)b * N + n) * r + i] = __float2bfloat16_rn(__int_as_float(0x7fc00000));
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) ptx::tmem_dealloc(tmem, 2 * acc_cols);
}

template <int D>
cudaError_t launch_d(int B, int N, int r, const void* H, const float* V, void* US, cudaStream_t st) {
  using Cfg = UsCfg<D>;
  const GramPlan plan = slice_plan(B, N);
  CUtensorMap tmap;
  if (!encode_tmap_bf16_3d(&tmap, H, D, (uint64_t)N, (uint64_t)B, (uint64_t)D * 2, (uint64_t)N * D * 2, 64,
                           kTileRows))
    return cudaErrorInvalidValue;
  const size_t smem = Cfg::smem((r + 15) & ~15);
  cudaError_t e = cudaFuncSetAttribute(project_us_umma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)Cfg::smem(kMaxCols));
  if (e != cudaSuccess) return e;
  const dim3 grid(plan.splits, B), block(kThreads);
  project_us_umma_kernel<D><<<grid, block, smem, st>>>(tmap, V, static_cast<__nv_bfloat16*>(US), N, r,
                                                           plan.chunk_tiles * kTileRows);
  return cudaGetLastError();
}

}  // namespace

bool project_us_umma_supported(int N, int d, int r, solar_dtype_t dt) {
  return dt == SOLAR_BF16 && (d == 64 || d == 128) && N >= kTileRows && r >= 1 && r <= kMaxCols;
}

cudaError_t launch_project_us_umma(int B, int N, int d, int r, const void* H, const float* V, void* US,
                                   cudaStream_t st) {
  return d == 64 ? launch_d<64>(B, N, r, H, V, US, st) : launch_d<128>(B, N, r, H, V, US, st);
}

}  // namespace solar
