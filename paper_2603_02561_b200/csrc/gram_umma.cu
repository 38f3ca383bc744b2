// Streaming Gram pass on the tensor cores (bf16 storage, d = 64 or 128):
//   P[b,s] = sum_{n in slice s} h_n h_n^T,   G_b = H_b^T H_b = sum_s P[b,s]
// (G_b is the matrix whose eigenvectors are V of Eq. 9).
//
// One CTA per (user, slice).  A single thread streams the slice's 128-row tiles of H
// through a ring of shared-memory stages with TMA (128-byte swizzle, zero fill past row
// N, so ragged tails add nothing); a single thread issues tcgen05.mma with the SAME tile
// as both operands -- H^T as an MN-major A and H as an MN-major B, K = the 128 rows --
// accumulating the d x d result in tensor memory.  H is read from HBM exactly once and never
// passes through registers.
//
// The CTAs of up to eight slices of a user form a thread-block cluster: each lays its
// accumulator down in its own shared memory, and after a cluster barrier every CTA adds up
// one share of the matrix over all of them through distributed shared memory (plain loads, in
// rank order: the sum is reproducible) and stores it.  A user so leaves splits / cluster
// partial matrices in global memory -- one in the usual case -- instead of one per slice.
#include "sm100_ptx.cuh"
#include "solar_internal.cuh"

namespace solar {

namespace {

constexpr int kTileRows = kGramTileRows;   // 128 rows of H per stage
constexpr int kErrProducer = 0x11, kErrMma = 0x12, kErrEpilogue = 0x13;

template <int D> struct GramCfg {
  static constexpr int BOXES = D / 64;                       // 64-column TMA boxes per tile
  static constexpr int BOX_BYTES = kTileRows * 128;          // 16 KB: 128 rows x 64 bf16
  static constexpr int TILE_BYTES = BOXES * BOX_BYTES;
  // Three 16 KB stages at d = 64 (four of 32 KB at d = 128).  Alone a deeper ring changes nothing
  // (7.9 us either way); with many requests in flight the CTA's shared-memory footprint is what
  // counts -- the step takes 8.87 / 8.63 / 8.49 / 8.67 us with 5 / 4 / 3 / 2 stages on the
  // 16 x 10240 x 64 serving shape -- because the Gram, eigensolver and attention CTAs of different
  // requests share every SM's 227 KB.
  static constexpr int STAGES = (D == 64) ? 3 : 4;
  static constexpr size_t SMEM = (size_t)STAGES * TILE_BYTES + 1024;   // + slack to align to 1024
  static constexpr uint32_t IDESC = ptx::umma_idesc_bf16(D, D, true, true);
};

template <int D>
__global__ void __launch_bounds__(128, 1)
gram_umma_kernel(const __grid_constant__ CUtensorMap tmap, float* __restrict__ gpart,
                 int* __restrict__ status, int N, int chunk_rows, int splits, int cluster) {
  using Cfg = GramCfg<D>;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ __align__(8) uint64_t accum_bar;
  __shared__ uint32_t s_tmem;
  __shared__ int s_err;

  const int b = blockIdx.y, s = blockIdx.x;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int row0 = s * chunk_rows;
  const int row1 = min(N, row0 + chunk_rows);
  const int ntiles = (row1 - row0 + kTileRows - 1) / kTileRows;   // >= 1 by construction of the plan

  if (tid == 0) {
    s_err = 0;
    for (int i = 0; i < STAGES; ++i) { ptx::mbar_init(&full_bar[i], 1); ptx::mbar_init(&empty_bar[i], 1); }
    ptx::mbar_init(&accum_bar, 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmap);
  }
  if (warp == 1) ptx::tmem_alloc(&s_tmem, D);
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem = s_tmem;
  volatile int* err = &s_err;

  if (warp == 0 && lane == 0) {
    // ---- producer: one TMA tile per stage ------------------------------------------
    // H is the caller's: whatever wrote it earlier on the stream must have completed before the
    // first tile is fetched (the set-up above did overlap that kernel's tail)
    pdl_wait();
    int issued = 0;
    for (int t = 0; t < ntiles; ++t) {
      const int st = t % STAGES;
      if (t >= STAGES && !ptx::mbar_wait(&empty_bar[st], ((t / STAGES) - 1) & 1, err, kErrProducer)) break;
      ptx::mbar_arrive_expect_tx(&full_bar[st], Cfg::TILE_BYTES);
#pragma unroll
      for (int x = 0; x < Cfg::BOXES; ++x)
        ptx::tma_load_3d(tiles + (size_t)st * Cfg::TILE_BYTES + x * Cfg::BOX_BYTES, &tmap, &full_bar[st],
                         x * 64, row0 + t * kTileRows, b);
      issued = t + 1;
    }
    if (*err != 0) {
      // a wait ran out somewhere: let the copies still in flight land before the CTA leaves
      for (int t = max(0, issued - STAGES); t < issued; ++t) {
        int dummy = 0;
        ptx::mbar_wait(&full_bar[t % STAGES], (t / STAGES) & 1, &dummy, 0);
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer: G += tile^T tile, 8 steps of K = 16 rows ------------------------
    for (int t = 0; t < ntiles; ++t) {
      const int st = t % STAGES;
      if (!ptx::mbar_wait(&full_bar[st], (t / STAGES) & 1, err, kErrMma)) break;
      ptx::tc_fence_after_sync();
      const uint32_t base = ptx::smem_u32(tiles + (size_t)st * Cfg::TILE_BYTES);
#pragma unroll
      for (int ks = 0; ks < kTileRows / 16; ++ks) {
        // 16 rows = two 8-row swizzle atoms of 1024 B; 64-column blocks are BOX_BYTES apart
        const uint64_t desc = ptx::umma_smem_desc(base + ks * 2048, Cfg::BOX_BYTES, 1024);
        ptx::umma_bf16_ss(tmem, desc, desc, Cfg::IDESC, (t | ks) != 0);
      }
      ptx::umma_commit(&empty_bar[st]);      // the stage is free once these MMAs have read it
    }
    ptx::umma_commit(&accum_bar);            // arrives when the whole accumulation is done
  }
  __syncwarp();

  // ---- epilogue: tensor memory -> shared memory -> sum over the cluster -> global ----------
  const bool done = ptx::mbar_wait(&accum_bar, 0, err, kErrEpilogue);
  pdl_trigger();       // only the epilogue is left: the next kernel may start launching
  __syncwarp();
  ptx::tc_fence_after_sync();
  // the accumulator as a row-major fp32 matrix over the ring (every tile has been consumed);
  // the row pitch D + 4 keeps the 16-byte stores of a warp's 32 rows off each other's banks
  constexpr int LDR = D + 4;
  float* red = reinterpret_cast<float*>(tiles);
  static_assert((size_t)D * LDR * sizeof(float) <= (size_t)STAGES * Cfg::TILE_BYTES, "the matrix fits over the ring");
  if (done && *err == 0) {
    // M = 128: accumulator row i sits in lane i.  M = 64: rows 16q .. 16q+15 sit in lanes
    // 32q .. 32q+15 (each warp reaches only its own 32-lane quarter).
    const int row = (D == 128) ? (warp * 32 + lane) : (warp * 16 + lane);
    const bool has_row = (D == 128) || (lane < 16);
#pragma unroll
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t v[32];
      ptx::tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + c0, v);
      ptx::tmem_ld_wait();
      if (has_row) {
        float4* dst = reinterpret_cast<float4*>(red + (size_t)row * LDR + c0);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                               __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
      }
    }
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) ptx::tmem_dealloc(tmem, D);
  if (tid == 0) status[b * splits + s] = (s_err == 0) ? kGramStatusOk : s_err;
  // Every CTA of the cluster reaches the two cluster barriers, whatever happened above (a lost
  // wait is reported through the status word; the sum of that user is then not used).
  if (cluster > 1) ptx::cluster_sync();
  // nothing is written before the previous kernel on the stream (it may still be reading this
  // workspace) has completed
  pdl_wait();
  {
    const int rank = s % cluster;
    float* out = gpart + ((size_t)b * (splits / cluster) + s / cluster) * D * D;
    // this CTA's share of the matrix: 16-byte elements rank, rank + cluster, ...
    for (int e = rank * 128 + tid; e < D * D / 4; e += cluster * 128) {
      const int row = e / (D / 4), c4 = e % (D / 4);
      const float* src = red + (size_t)row * LDR + 4 * c4;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (cluster > 1) {
        for (int q = 0; q < cluster; ++q) {
          const float4 t = ptx::ld_cluster_f4(src, q);
          acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
      } else {
        acc = *reinterpret_cast<const float4*>(src);
      }
      reinterpret_cast<float4*>(out)[e] = acc;
    }
  }
  if (cluster > 1) ptx::cluster_sync();      // nobody leaves while its matrix is still being read
}

template <int D>
cudaError_t launch_d(int B, int N, const void* H, float* gpart, int* status, const GramPlan& plan,
                     cudaStream_t st) {
  using Cfg = GramCfg<D>;
  CUtensorMap tmap;
  if (!encode_tmap_bf16_3d(&tmap, H, D, (uint64_t)N, (uint64_t)B, (uint64_t)D * 2, (uint64_t)N * D * 2, 64,
                           kTileRows))
    return cudaErrorInvalidValue;
  static bool limits_set[kMaxDevicesCached] = {};
  const cudaError_t e = set_kernel_limits(reinterpret_cast<const void*>(&gram_umma_kernel<D>), Cfg::SMEM, limits_set);
  if (e != cudaSuccess) return e;
  const dim3 grid(plan.splits, B), block(128);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = Cfg::SMEM; cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = (unsigned)plan.cluster; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = plan.cluster > 1 ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, gram_umma_kernel<D>, tmap, gpart, status, N, plan.chunk_tiles * kTileRows,
                            plan.splits, plan.cluster);
}

}  // namespace

bool gram_umma_supported(int N, int d, solar_dtype_t dt) {
  return dt == SOLAR_BF16 && (d == 64 || d == 128) && N >= kTileRows;
}

cudaError_t launch_gram_umma(int B, int N, int d, const void* H, float* gpart, int* status,
                             const GramPlan& plan, cudaStream_t st) {
  return d == 64 ? launch_d<64>(B, N, H, gpart, status, plan, st)
                 : launch_d<128>(B, N, H, gpart, status, plan, st);
}

}  // namespace solar
