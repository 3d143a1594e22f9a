// The dense weight gradient of the layer step (straight-through estimator), D[i, j] = sum_t dY[t, i] X[t, j], on
// tcgen05.mma: CTA pairs for layers of more than 128 rows, single CTAs below, split-K work items for small outputs,
// and the implicit form for 3x3 convolutions.  Structure and waits as in spmm_sm100.cu.
#include "gemm_common.cuh"

namespace bimask {

namespace {

// ------------------------------------------------------------------------------------------
// Dense weight gradient on CTA pairs, persistent.  D[i, j] = sum_t dY[t, i] X[t, j]: both
// operands are read MN-major straight from the row-major activations (no transpose pass).  A
// pair owns a 256 x 256 tile; each CTA loads its 128 rows of dY^T and 128 of the 256 columns of
// X per stage (32 KB), the leader issues tcgen05.mma.cta_group::2, and the 512 tensor-memory
// columns hold TWO accumulators, so the epilogue of one tile (tensor memory -> registers ->
// 128-byte runs of fp32 in global memory) overlaps the main loop of the next.
// Work items are (tile, k-split) pairs; with more than one split the partial sums go to scratch.
// ------------------------------------------------------------------------------------------
// Epilogue of both kernels.  The accumulator holds D[row][column] with row = tensor-memory lane, and dW is
// row-major, so a lane owns 128 contiguous bytes per 32-column chunk -- but stored from registers every instruction
// of a warp would touch 32 different lines.  Instead the four draining warps write the chunk (128 rows x 128 bytes)
// into one of two staging tiles in the 128-byte-swizzled layout (16-byte unit index XOR row mod 8: conflict-free
// 16-byte shared stores) and a fifth warp's elected thread sends the tile off with one tensor store (TMA) of a
// 32 x 128 box; rows and columns outside dW are clipped by the tensor map.  Two mbarriers per tile hand it back and
// forth: staged[t] (four arrivals, one per draining warp) and freed[t] (the store thread, once the store has read
// the tile).  `u`: the CTA's chunk counter, carried from work item to work item (tile u % 2).
constexpr int WGRAD_THREADS = GEMM_THREADS + 32;                 // + the store warp
constexpr int WGRAD_STAGING_BYTES = 2 * 16384;
constexpr uint32_t WGRAD_EPI_BAR_OFFSET = 160;                   // staged[2], freed[2] inside the barrier area, past the kernels' own barriers and words

__device__ __forceinline__ void wgrad_epi_bars_init(uint32_t bar_area) {
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    ptx::mbar_init(bar_area + WGRAD_EPI_BAR_OFFSET + 8u * t, 4);
    ptx::mbar_init(bar_area + WGRAD_EPI_BAR_OFFSET + 8u * (2 + t), 1);
  }
}

// One draining warp's share of an accumulator: lane quadrant q, columns 0..255 in eight chunks.  `acc`: the
// accumulator's tensor-memory address with the quadrant's lane offset.  release() is called once the last chunk has
// been read from tensor memory.  Returns false when a wait ran out of budget.
template <typename Release>
__device__ __forceinline__ bool wgrad_drain(uint32_t acc, uint32_t stg, uint32_t bar_area, uint32_t& u, int q, int lane,
                                            volatile int* abort_flag, Release&& release) {
  const uint32_t bars = bar_area + WGRAD_EPI_BAR_OFFSET;
  const uint32_t row = (uint32_t)(32 * q + lane);
  const uint32_t row_addr = stg + row * 128u;
  const uint32_t sw = row & 7u;
  bool ok = true;
  auto stage = [&](const uint32_t (&r)[32]) {
    const uint32_t slot = u & 1u, use = u >> 1;
    ++u;
    if (use > 0 && ok) ok = ptx::mbar_wait_bounded(bars + 8u * (2 + slot), (use - 1u) & 1u, abort_flag, WAIT_BUDGET);
#pragma unroll
    for (uint32_t j = 0; j < 8; ++j)
      ptx::st_shared_v4(row_addr + slot * 16384u + ((j ^ sw) << 4), r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(bars + 8u * slot);
  };
  uint32_t ra[32], rb[32];
  ptx::tmem_ld_32x32(acc, ra);
#pragma unroll 1
  for (int c = 0; c < 8; c += 2) {
    ptx::tmem_ld_wait();
    ptx::tmem_ld_32x32(acc + 32 * (c + 1), rb);
    stage(ra);
    ptx::tmem_ld_wait();
    if (c + 2 < 8) ptx::tmem_ld_32x32(acc + 32 * (c + 2), ra); else release();
    stage(rb);
  }
  return ok;
}

// The store thread's side for one work item: first row m0 of the CTA's 128, first column n0 of the tile's 256.
__device__ __forceinline__ bool wgrad_store_item(const CUtensorMap* tmapD, uint32_t stg, uint32_t bar_area, uint32_t& u, int m0,
                                                 int n0, int split, int Mdim, int Ndim, volatile int* abort_flag) {
  const uint32_t bars = bar_area + WGRAD_EPI_BAR_OFFSET;
  for (int c = 0; c < 8; ++c) {
    const uint32_t slot = u & 1u, use = u >> 1;
    if (!ptx::mbar_wait_bounded(bars + 8u * slot, use & 1u, abort_flag, WAIT_BUDGET)) return false;
    const int nb = n0 + 32 * c;
    if (nb < Ndim && m0 < Mdim) ptx::tma_store_4d(tmapD, nb, m0, split, 0, stg + slot * 16384u);
    ptx::bulk_commit();
    if (u > 0) {
      ptx::bulk_wait_read<1>();
      ptx::mbar_arrive(bars + 8u * (2 + ((u - 1u) & 1u)));
    }
    ++u;
  }
  return true;
}

template <int STAGES>
struct WgradCfg {
  static constexpr int A_BYTES = 16384, B_BYTES = 16384;     // 128 x 64 bf16 each, as two 64-wide boxes
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + WGRAD_STAGING_BYTES + 1024 + 256;
};

// CONV: k tile kt is pixel box kt (64 pixels) of the NHWC tensors; the dy operand is that box, the
// x operand the same box shifted by the filter tap its 64 columns of dW belong to.
template <int STAGES, bool CONV>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(WGRAD_THREADS, 1)
wgrad_pair_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                  const __grid_constant__ CUtensorMap tmapD, const GemmParams p, int splits) {
  pdl_launch_dependents();
  using C = WgradCfg<STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t staging = base + STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = staging + WGRAD_STAGING_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tmem_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tmem_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + WGRAD_STAGING_BYTES + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int num_items = num_tiles * splits;
  const int k_tiles_total = (p.Kdim + 63) / 64;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tmem_full_bar(b), 1);
      ptx::mbar_init(tmem_empty_bar(b), 8);
    }
    wgrad_epi_bars_init(bar_base);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    ptx::prefetch_tmap(&tmapD);
  }
  if (warp == 1) {
    ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), C::TMEM_COLS);
    ptx::tmem_relinquish_pair();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                            // barriers, tensor memory and tensor-map prefetch needed no global memory

  // item -> (tile, split) -> coordinates; identical in every role
  auto item_coords = [&](int item, int& m0, int& n0, int& kt0, int& nkt, int& split) {
    const int tile = item % num_tiles;
    split = item / num_tiles;
    int tile_m, tile_n;
    raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
    m0 = (2 * tile_m + (int)rank) * 128;
    n0 = tile_n * 256;
    kt0 = split * p.k_tiles_per_split;
    nkt = min(k_tiles_total, kt0 + p.k_tiles_per_split) - kt0;
  };

  if (warp == 0) {
    if (ptx::elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = cluster_id; item < num_items && ok; item += num_clusters) {
        int m0, n0, kt0, nkt, split;
        item_coords(item, m0, n0, kt0, nkt, split);
        for (int kt = kt0; kt < kt0 + nkt; ++kt, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + C::A_BYTES;
          const uint32_t bar = ptx::mapa(full_bar(s), 0);
          if (rank == 0) ptx::mbar_expect_tx(full_bar(s), 2 * C::STAGE_BYTES);
          if (CONV) {
            int cw0, ch0, cn0;
            conv_box_origin(p.conv, kt, cw0, ch0, cn0);
            ptx::tma_load_4d_pair(a_s, &tmapA, m0, cw0, ch0, cn0, bar);
            ptx::tma_load_4d_pair(a_s + 8192, &tmapA, m0 + 64, cw0, ch0, cn0, bar);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const int j = n0 + 128 * (int)rank + 64 * q;           // first of 64 columns of dW: one tap, 64 channels
              const bool valid = j < p.Ndim;
              const int tap = j / p.conv.CB;
              ptx::tma_load_4d_pair(b_s + q * 8192, &tmapB, valid ? j - tap * p.conv.CB : 0, p.conv.stride * cw0 + tap % 3 - 1,
                                    p.conv.stride * ch0 + tap / 3 - 1, valid ? cn0 : p.conv.NB, bar);
            }
            continue;
          }
          ptx::tma_load_2d_pair(a_s, &tmapA, m0, kt * 64, bar);
          ptx::tma_load_2d_pair(a_s + 8192, &tmapA, m0 + 64, kt * 64, bar);
          ptx::tma_load_2d_pair(b_s, &tmapB, n0 + 128 * (int)rank, kt * 64, bar);
          ptx::tma_load_2d_pair(b_s + 8192, &tmapB, n0 + 128 * (int)rank + 64, kt * 64, bar);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::idesc_bf16(256, 256, true, true, false);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int item = cluster_id; item < num_items && ok; item += num_clusters, ++tcount) {
        int m0, n0, kt0, nkt, split;
        item_coords(item, m0, n0, kt0, nkt, split);
        const uint32_t buf = tcount & 1u;
        if (!ptx::mbar_wait_bounded(tmem_empty_bar(buf), ((tcount >> 1) & 1u) ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        ptx::tc_fence_after();
        const uint32_t acc = tmem_base + 256u * buf;
        for (int k = 0; k < nkt; ++k, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + C::A_BYTES;
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t ad = ptx::smem_desc(a_s + kb * 2048, 8192, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + kb * 2048, 8192, 1024, 2);
            ptx::mma_dense_pair(acc, ad, bd, idesc, (k | kb) != 0);
          }
          ptx::tc_commit_pair(empty_bar(s), 3);
        }
        if (ok) ptx::tc_commit_pair(tmem_full_bar(buf), 3);
      }
    }
  } else if (warp < 6) {
    const int q = warp & 3;
    uint32_t tcount = 0, u = 0;
    for (int item = cluster_id; item < num_items; item += num_clusters, ++tcount) {
      const uint32_t buf = tcount & 1u;
      if (!ptx::mbar_wait_bounded(tmem_full_bar(buf), (tcount >> 1) & 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
      const uint32_t release_bar = ptx::mapa(tmem_empty_bar(buf), 0);
      if (!wgrad_drain(tmem_base + 256u * buf + ((uint32_t)(32 * q) << 16), staging, bar_base, u, q, lane, abort_flag, [&] {
            ptx::tc_fence_before();                        // accumulator drained: release it
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_cluster(release_bar);
          })) {
        *abort_flag = 1;
        break;
      }
    }
  } else {
    // store thread: the same walk over the work items as the draining warps
    if (ptx::elect_one()) {
      uint32_t u = 0;
      for (int item = cluster_id; item < num_items; item += num_clusters) {
        int m0, n0, kt0, nkt, split;
        item_coords(item, m0, n0, kt0, nkt, split);
        if (!wgrad_store_item(&tmapD, staging, bar_base, u, m0, n0, split, p.Mdim, p.Ndim, abort_flag)) { *abort_flag = 1; break; }
      }
      ptx::bulk_wait_read<0>();                            // shared memory must outlive the stores that read it
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status_word, (int32_t)BIMASK_ETIMEOUT);
  ptx::cluster_sync();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------
// Dense weight gradient, one CTA per 128 x 256 tile: for layers of at most 128 output rows the
// pair kernel above would leave half of every 256-row MMA tile empty.  Same pipeline without the
// cluster: 16 KB of dY^T and 32 KB of X per stage, tcgen05.mma.cta_group::1 128 x 256 x 16, two
// accumulators in tensor memory, persistent over (tile, k-split) work items.
// ------------------------------------------------------------------------------------------
template <int STAGES>
struct WgradSingleCfg {
  static constexpr int A_BYTES = 16384, B_BYTES = 32768;     // 128 and 256 columns x 64 tokens, 64-wide boxes
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + WGRAD_STAGING_BYTES + 1024 + 256;
};

template <int STAGES, bool CONV>
__global__ void __launch_bounds__(WGRAD_THREADS, 1)
wgrad_single_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                    const __grid_constant__ CUtensorMap tmapD, const GemmParams p, int splits) {
  pdl_launch_dependents();
  using C = WgradSingleCfg<STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t staging = base + STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = staging + WGRAD_STAGING_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tmem_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tmem_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + WGRAD_STAGING_BYTES + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = p.tiles_m * p.tiles_n;            // tiles_m counts 128-row tiles
  const int num_items = num_tiles * splits;
  const int k_tiles_total = (p.Kdim + 63) / 64;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tmem_full_bar(b), 1);
      ptx::mbar_init(tmem_empty_bar(b), 4);               // four epilogue warps
    }
    wgrad_epi_bars_init(bar_base);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    ptx::prefetch_tmap(&tmapD);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                            // barriers, tensor memory and tensor-map prefetch needed no global memory

  auto item_coords = [&](int item, int& m0, int& n0, int& kt0, int& nkt, int& split) {
    const int tile = item % num_tiles;
    split = item / num_tiles;
    int tile_m, tile_n;
    raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
    m0 = tile_m * 128;
    n0 = tile_n * 256;
    kt0 = split * p.k_tiles_per_split;
    nkt = min(k_tiles_total, kt0 + p.k_tiles_per_split) - kt0;
  };

  if (warp == 0) {
    if (ptx::elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x) {
        int m0, n0, kt0, nkt, split;
        item_coords(item, m0, n0, kt0, nkt, split);
        for (int kt = kt0; kt < kt0 + nkt; ++kt, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + C::A_BYTES;
          ptx::mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
          if (CONV) {
            int cw0, ch0, cn0;
            conv_box_origin(p.conv, kt, cw0, ch0, cn0);
            ptx::tma_load_4d(a_s, &tmapA, m0, cw0, ch0, cn0, full_bar(s));
            ptx::tma_load_4d(a_s + 8192, &tmapA, m0 + 64, cw0, ch0, cn0, full_bar(s));
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int j = n0 + 64 * q;                   // first of 64 columns of dW: one tap, 64 channels
              const bool valid = j < p.Ndim;
              const int tap = j / p.conv.CB;
              ptx::tma_load_4d(b_s + q * 8192, &tmapB, valid ? j - tap * p.conv.CB : 0, p.conv.stride * cw0 + tap % 3 - 1, p.conv.stride * ch0 + tap / 3 - 1,
                               valid ? cn0 : p.conv.NB, full_bar(s));
            }
            continue;
          }
          ptx::tma_load_2d(a_s, &tmapA, m0, kt * 64, full_bar(s));
          ptx::tma_load_2d(a_s + 8192, &tmapA, m0 + 64, kt * 64, full_bar(s));
#pragma unroll
          for (int q = 0; q < 4; ++q) ptx::tma_load_2d(b_s + q * 8192, &tmapB, n0 + 64 * q, kt * 64, full_bar(s));
        }
      }
    }
  } else if (warp == 1) {
    if (ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::idesc_bf16(128, 256, true, true, false);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < num_items && ok; item += gridDim.x, ++tcount) {
        int m0, n0, kt0, nkt, split;
        item_coords(item, m0, n0, kt0, nkt, split);
        const uint32_t buf = tcount & 1u;
        if (!ptx::mbar_wait_bounded(tmem_empty_bar(buf), ((tcount >> 1) & 1u) ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        ptx::tc_fence_after();
        const uint32_t acc = tmem_base + 256u * buf;
        for (int k = 0; k < nkt; ++k, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + C::A_BYTES;
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t ad = ptx::smem_desc(a_s + kb * 2048, 8192, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + kb * 2048, 8192, 1024, 2);
            ptx::mma_dense(acc, ad, bd, idesc, (k | kb) != 0);
          }
          ptx::tc_commit(empty_bar(s));
        }
        if (ok) ptx::tc_commit(tmem_full_bar(buf));
      }
    }
  } else if (warp < 6) {
    const int q = warp & 3;
    uint32_t tcount = 0, u = 0;
    for (int item = blockIdx.x; item < num_items; item += gridDim.x, ++tcount) {
      const uint32_t buf = tcount & 1u;
      if (!ptx::mbar_wait_bounded(tmem_full_bar(buf), (tcount >> 1) & 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
      if (!wgrad_drain(tmem_base + 256u * buf + ((uint32_t)(32 * q) << 16), staging, bar_base, u, q, lane, abort_flag, [&] {
            ptx::tc_fence_before();                        // accumulator drained: release it
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_relaxed(tmem_empty_bar(buf));
          })) {
        *abort_flag = 1;
        break;
      }
    }
  } else {
    // store thread: the same walk over the work items as the draining warps
    if (ptx::elect_one()) {
      uint32_t u = 0;
      for (int item = blockIdx.x; item < num_items; item += gridDim.x) {
        int m0, n0, kt0, nkt, split;
        item_coords(item, m0, n0, kt0, nkt, split);
        if (!wgrad_store_item(&tmapD, staging, bar_base, u, m0, n0, split, p.Mdim, p.Ndim, abort_flag)) { *abort_flag = 1; break; }
      }
      ptx::bulk_wait_read<0>();                            // shared memory must outlive the stores that read it
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status_word, (int32_t)BIMASK_ETIMEOUT);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// Sum of split-K partials: out[e] = sum_s part[s][e], one thread per float4 -- for outputs large enough to fill
// the GPU that way.
__global__ void splitk_reduce_kernel(const float4* __restrict__ part, int splits, long long n4,
                                     float4* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += (long long)gridDim.x * blockDim.x) {
    float4 acc = part[e];
    for (int s = 1; s < splits; ++s) {
      const float4 v = part[(long long)s * n4 + e];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    out[e] = acc;
  }
}

// The same sum for small outputs with many splits (a 64 x 576 gradient cut 49 ways): a CTA covers 32 consecutive
// float4 columns, its eight warps take the splits in turn (warp w: splits w, w + 8, ...) and the eight partial sums
// are added in warp order through shared memory.
__global__ void __launch_bounds__(256)
splitk_reduce_wide_kernel(const float4* __restrict__ part, int splits, long long n4, float4* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float4 red[8][32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (long long e0 = (long long)blockIdx.x * 32; e0 < n4; e0 += (long long)gridDim.x * 32) {
    const long long e = e0 + lane;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (e < n4) {
#pragma unroll 4
      for (int sp = w; sp < splits; sp += 8) {
        const float4 v = __ldg(part + (long long)sp * n4 + e);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
    }
    red[w][lane] = acc;
    __syncthreads();
    if (w == 0 && e < n4) {
#pragma unroll
      for (int k = 1; k < 8; ++k) {
        const float4 v = red[k][lane];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      out[e] = acc;
    }
    __syncthreads();
  }
}

}  // namespace

// Adds up the split-K partial results into dW.
static int launch_splitk_reduce(const float* partials, int splits, long long n4, float* dW, cudaStream_t s) {
  const float4* part = reinterpret_cast<const float4*>(partials);
  float4* out = reinterpret_cast<float4*>(dW);
  if (n4 >= 148 * 1024 || splits < 8) {
    long long blocks = (n4 + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    BIMASK_CUDA_OK(launch_pdl(splitk_reduce_kernel, (unsigned)blocks, 256, 0, s, part, splits, n4, out));
  } else {
    const long long blocks = (n4 + 31) / 32;               // < 148 * 32
    BIMASK_CUDA_OK(launch_pdl(splitk_reduce_wide_kernel, (unsigned)blocks, 256, 0, s, part, splits, n4, out));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// Split-K plan of the dense product for a reduction of k_tiles 64-deep tiles.
static bool wgrad_uses_single(int I) { return I <= 128; }       // one 128-row tile: no CTA pairs

static void wgrad_plan_k(int k_tiles, int I, int J, int* splits, int* k_tiles_per_split) {
  const bool single = wgrad_uses_single(I);
  const int tiles = single ? (J + 255) / 256 : (((I + 127) / 128 + 1) / 2) * ((J + 255) / 256);   // 128 / 256 x 256 tiles
  const int workers = single ? 148 : 74;                          // CTAs or CTA pairs
  int sp = 1;
  if (tiles < workers) {
    sp = workers / tiles;                                         // one round of work items over the workers
    const int max_by_k = k_tiles / 8 > 0 ? k_tiles / 8 : 1;        // at least 8 k tiles per split
    if (sp > max_by_k) sp = max_by_k;
    if (sp > 64) sp = 64;
  }
  int per = (k_tiles + sp - 1) / sp;
  sp = (k_tiles + per - 1) / per;
  *splits = sp; *k_tiles_per_split = per;
}

// Launches the pair or the single kernel for a prepared problem.  LIGHT: four (three) stages instead of six (four),
// about 160 KB of shared memory instead of 225 KB: the layers that the step spreads over several streams keep every SM
// for tens of microseconds with one persistent CTA, and only with room left beside it can the short mask and search
// kernels of the same step run at the same time instead of queueing behind it; their reductions are short enough
// for the shallower ring to cost nothing.
template <bool LIGHT, bool CONV>
static int launch_wgrad_kernel(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& td, GemmParams& p, int I,
                               int splits, cudaStream_t s) {
  constexpr int PAIR_STAGES = LIGHT ? 4 : 6, SINGLE_STAGES = LIGHT ? 3 : 4;
  const int sms = sm_count();
  int rc;
  if (wgrad_uses_single(I)) {
    using C1 = WgradSingleCfg<SINGLE_STAGES>;
    auto kern1 = wgrad_single_kernel<SINGLE_STAGES, CONV>;
    if ((rc = set_smem_attr(kern1, C1::SMEM_BYTES)) != BIMASK_OK) return rc;
    p.tiles_m = 1;
    const int items = p.tiles_n * splits;
    BIMASK_CUDA_OK(launch_pdl(kern1, items < sms ? items : sms, WGRAD_THREADS, C1::SMEM_BYTES, s, ta, tb, td, p, splits));
  } else {
    using C = WgradCfg<PAIR_STAGES>;
    auto kern = wgrad_pair_kernel<PAIR_STAGES, CONV>;
    if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
    p.tiles_m = ((I + 127) / 128 + 1) / 2;
    const int items = p.tiles_m * p.tiles_n * splits;
    const int clusters = items < sms / 2 ? items : sms / 2;
    BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, WGRAD_THREADS, C::SMEM_BYTES, s, ta, tb, td, p, splits));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}
static bool wgrad_is_light(double tokens, int I, int J) { return 2.0 * tokens * I * J < 1e11; }

// The same for the implicit convolution: one k tile per 64-pixel box.
// H, W: the input image; the k tiles are boxes of OUTPUT pixels.
static ConvGeom conv_wgrad_geom(int NB, int H, int W, int C, int stride) {
  ConvGeom g{};
  g.mode = 1; g.NB = NB; g.CB = C; g.stride = stride;
  g.H = (H - 1) / stride + 1; g.W = (W - 1) / stride + 1;
  conv_boxes(g, 64);
  return g;
}

void wgrad_conv_plan(int NB, int H, int W, int C, int I, int stride, int* splits, int* k_tiles_per_split) {
  const ConvGeom g = conv_wgrad_geom(NB, H, W, C, stride);
  wgrad_plan_k(g.tiles_w * g.tiles_h * ((NB + g.nb - 1) / g.nb), I, 9 * C, splits, k_tiles_per_split);
}

// dW[i, tap*C + c] = sum over output pixels of dy[pixel, i] x[stride * pixel + tap, c] without a column matrix
// (C % 64 == 0).  partials: splits * I * 9C floats when wgrad_conv_plan gives more than one split.
int launch_wgrad_conv(const uint16_t* dy, const uint16_t* x, int NB, int H, int W, int C, int I, int stride, float* dW,
                      float* partials, int32_t* status_word, cudaStream_t s, cudaStream_t reduce_stream, cudaEvent_t product_done) {
  const ConvGeom g = conv_wgrad_geom(NB, H, W, C, stride);
  const int boxes = g.tiles_w * g.tiles_h * ((NB + g.nb - 1) / g.nb);
  const int J = 9 * C;
  int splits, per;
  wgrad_plan_k(boxes, I, J, &splits, &per);
  CUtensorMap ta, tb, td;
  int rc;
  if ((rc = make_tmap_nhwc_load(&ta, dy, I, g.W, g.H, NB, g.wb, g.hb, g.nb)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_nhwc_load(&tb, x, C, W, H, NB, g.wb, g.hb, g.nb, stride)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_f32_store(&td, splits > 1 ? partials : dW, (uint64_t)J, (uint64_t)I, (uint64_t)splits)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv = g;
  p.hw_meta = nullptr; p.tiles_k_meta = 0;
  p.Mdim = I; p.Ndim = J; p.Kdim = boxes * 64;
  p.k_tiles_per_split = per;
  p.out = splits > 1 ? partials : dW;
  p.status_word = status_word;
  p.tiles_n = (J + 255) / 256;
  p.raster_group = 8;
  rc = wgrad_is_light((double)boxes * 64, I, J) ? launch_wgrad_kernel<true, true>(ta, tb, td, p, I, splits, s)
                                                  : launch_wgrad_kernel<false, true>(ta, tb, td, p, I, splits, s);
  if (rc != BIMASK_OK) return rc;
  if (splits > 1) {
    const long long n4 = (long long)I * J / 4;
    if (reduce_stream && product_done) {
      BIMASK_CUDA_OK(cudaEventRecord(product_done, s));
      BIMASK_CUDA_OK(cudaStreamWaitEvent(reduce_stream, product_done, 0));
      s = reduce_stream;
    }
    if ((rc = launch_splitk_reduce(partials, splits, n4, dW, s)) != BIMASK_OK) return rc;
  }
  return BIMASK_OK;
}

// Split-K plan of the dense product, shared by the launcher and the workspace-size query.
void wgrad_plan(int T, int I, int J, int* n_tile, int* splits, int* k_tiles_per_split) {
  *n_tile = 256;
  wgrad_plan_k((T + 63) / 64, I, J, splits, k_tiles_per_split);
}

int launch_wgrad_impl(const uint16_t* dY, const uint16_t* X, int T, int I, int J, float* dW, float* partials,
                      int32_t* status_word, cudaStream_t s, cudaStream_t reduce_stream, cudaEvent_t product_done) {
  int nt, splits, per;
  wgrad_plan(T, I, J, &nt, &splits, &per);
  CUtensorMap ta, tb, td;
  int rc;
  if ((rc = make_tmap(&ta, dY, (uint64_t)I, (uint64_t)T, 64)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, X, (uint64_t)J, (uint64_t)T, 64)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_f32_store(&td, splits > 1 ? partials : dW, (uint64_t)J, (uint64_t)I, (uint64_t)splits)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv.mode = 0;
  p.hw_meta = nullptr; p.tiles_k_meta = 0;
  p.Mdim = I; p.Ndim = J; p.Kdim = T;
  p.k_tiles_per_split = per;
  p.out = splits > 1 ? partials : dW;
  p.status_word = status_word;
  p.tiles_n = (J + 255) / 256;
  p.raster_group = 8;
  rc = wgrad_is_light((double)T, I, J) ? launch_wgrad_kernel<true, false>(ta, tb, td, p, I, splits, s)
                                       : launch_wgrad_kernel<false, false>(ta, tb, td, p, I, splits, s);
  if (rc != BIMASK_OK) return rc;
  if (splits > 1) {
    const long long n4 = (long long)I * J / 4;
    if (reduce_stream && product_done) {
      BIMASK_CUDA_OK(cudaEventRecord(product_done, s));
      BIMASK_CUDA_OK(cudaStreamWaitEvent(reduce_stream, product_done, 0));
      s = reduce_stream;
    }
    if ((rc = launch_splitk_reduce(partials, splits, n4, dW, s)) != BIMASK_OK) return rc;
  }
  return BIMASK_OK;
}

}  // namespace bimask
