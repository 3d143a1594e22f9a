// The two 2:4 products of the layer step on the 5th-generation tensor cores (the third product, the dense
// weight gradient, is in wgrad_sm100.cu):
//   sparse forward    D[i, t] = sum_j A_f[i, j] X[t, j]        (Eq. 3;  A_f 2:4 along j)
//   sparse input grad D[l, t] = sum_k A'[l, k] dYp[t, k]       (Eq. 10; A' 2:4 along permuted k)
//
// All kernels are warp-specialised: a TMA producer thread fills a ring of shared-memory stages
// (operands in the 128-byte-swizzled layouts the tensor core reads directly), one thread issues
// tcgen05.mma.sp (the index metadata of the 2:4 operand is copied shared -> tensor memory with
// tcgen05.cp right before the MMAs that use it), accumulators live in tensor memory, eight
// epilogue warps drain them into swizzled staging tiles and two store warps send those off as
// tensor stores (drain_chunks_tma / store_chunks in gemm_common.cuh; the implicit convolution,
// whose tokens are pixels, writes from the draining warps: drain_chunks).  The large-shape kernels
// (spmm_pair2m_kernel, spmm_pair_persistent_kernel) run CTA pairs persistently; spmm_single_kernel
// is the one-CTA-per-tile form for operands of at most 128 rows or at most 128 tokens, and also
// takes a dense A operand (masked weights of a pattern the 2:4 format cannot hold).
//
// Every wait on an mbarrier carries a cycle budget: when it runs out the kernel writes
// BIMASK_ETIMEOUT to the caller's status word, all roles unwind, tensor memory is released and
// the kernel returns.
#include "gemm_common.cuh"

namespace bimask {

namespace {

// SPARSE = false: the same pipeline on a dense bf16 A operand (masked weights of a pattern the
// 2:4 format cannot hold): 128 x 128 A tile per stage as two 64-wide boxes, eight K = 16 MMAs.
// CONV: the token operand is fetched as shifted pixel boxes (see ConvGeom); N_TILE tokens = one box.
template <int N_TILE, int STAGES, bool SPARSE, bool CONV>
__global__ void __launch_bounds__(PAIR_THREADS, 1)
spmm_single_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                   const __grid_constant__ CUtensorMap tmapD, const GemmParams p) {
  pdl_launch_dependents();
  using C = Cfg<N_TILE, STAGES, SPARSE>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t staging = base + STAGES * C::STAGE_BYTES;      // epilogue staging, C::EPI_NT tiles of 8 KB per group of four warps
  const uint32_t bar_base = staging + epi_staging_bytes(C::EPI_NT);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bar_base + 8u * (2 * STAGES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + epi_staging_bytes(C::EPI_NT) + 8 * (2 * STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int tile_m, tile_n;
  raster((int)blockIdx.x, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
  const int m0 = tile_m * C::M_TILE;
  const int n0 = tile_n * N_TILE;
  const int k_tiles_total = (p.Kdim + C::K_TILE - 1) / C::K_TILE;
  int cw0 = 0, ch0 = 0, cn0 = 0;                       // CONV: origin of this tile's pixel box
  if (CONV) conv_box_origin(p.conv, tile_n, cw0, ch0, cn0);
  const int kt_begin = blockIdx.z * p.k_tiles_per_split;
  const int kt_end = min(k_tiles_total, kt_begin + p.k_tiles_per_split);
  const int num_kt = kt_end - kt_begin;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(tmem_full_bar, 1);
    epi_bars_init<C::EPI_NT>(bar_base);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    if (!CONV) ptx::prefetch_tmap(&tmapD);
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
  const uint32_t tmem_meta = tmem_base + N_TILE;     // 4 columns after the accumulator (multiple of 4)

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (ptx::elect_one()) {
      for (int it = 0; it < num_kt; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
        if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        const int kt = kt_begin + it;
        const uint32_t a_s = base + s * C::STAGE_BYTES;
        const uint32_t b_s = a_s + C::A_BYTES;
        ptx::mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
        if (SPARSE && CONV) {
          int a_col = kt * 64, a_row = m0, meta_row = tile_m, meta_kt = kt;
          if (p.conv.mode == 2) {
            const int tap = kt / p.conv.kt_per_tap;
            meta_kt = kt - tap * p.conv.kt_per_tap;
            a_col = meta_kt * 64;
            a_row = p.conv.tap_id[tap] * p.conv.rows_per_tap + m0;
            meta_row = a_row >> 7;
          }
          ptx::tma_load_2d(a_s, &tmapA, a_col, a_row, full_bar(s));
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            int c0, dw, dh;
            bool valid;
            conv_k_coords(p.conv, kt, q, p.Kdim, c0, dw, dh, valid);
            ptx::tma_load_4d(b_s + q * (N_TILE * 128), &tmapB, valid ? c0 : 0, p.conv.stride * cw0 + dw, p.conv.stride * ch0 + dh, valid ? cn0 : p.conv.NB,
                             full_bar(s));
          }
          {
            // 64 rows per tap (C = 64): every other tap starts in the middle of a 128-row metadata block; its rows
            // are that block's lanes 64..127 (the second KiB), which must land in lanes 0..63 of the tile.  The
            // tile's other 64 rows belong to another tap and are never stored: they get the block's other half.
            const uint8_t* blk = p.hw_meta + ((size_t)meta_row * p.tiles_k_meta + meta_kt) * 2048;
            if (a_row & 64) {
              ptx::bulk_load(b_s + C::B_BYTES, blk + 1024, 1024, full_bar(s));
              ptx::bulk_load(b_s + C::B_BYTES + 1024, blk, 1024, full_bar(s));
            } else {
              ptx::bulk_load(b_s + C::B_BYTES, blk, 2048, full_bar(s));
            }
          }
          continue;
        }
        if (SPARSE) {
          ptx::tma_load_2d(a_s, &tmapA, kt * 64, m0, full_bar(s));                    // 64 compressed x 128 rows
        } else {
          ptx::tma_load_2d(a_s, &tmapA, kt * 128, m0, full_bar(s));                   // k 0..63
          ptx::tma_load_2d(a_s + 16384, &tmapA, kt * 128 + 64, m0, full_bar(s));      // k 64..127
        }
        ptx::tma_load_2d(b_s, &tmapB, kt * 128, n0, full_bar(s));                     // k 0..63
        ptx::tma_load_2d(b_s + N_TILE * 128, &tmapB, kt * 128 + 64, n0, full_bar(s)); // k 64..127
        if (SPARSE)
          ptx::bulk_load(b_s + C::B_BYTES,
                         p.hw_meta + ((size_t)tile_m * p.tiles_k_meta + kt) * 2048, 2048, full_bar(s));
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::idesc_bf16(128, N_TILE, false, false, SPARSE);
      bool ok = true;
      for (int it = 0; it < num_kt && ok; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
        if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t a_s = base + s * C::STAGE_BYTES;
        const uint32_t b_s = a_s + C::A_BYTES;
        if constexpr (SPARSE) {
          ptx::tmem_cp_128x128b(tmem_meta, ptx::smem_desc(b_s + C::B_BYTES, 0, 128, 0));
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t ad = ptx::smem_desc(a_s + kb * 32, 16, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + (kb >> 1) * (N_TILE * 128) + (kb & 1) * 64, 16, 1024, 2);
            ptx::mma_sparse(tmem_base, ad, bd, tmem_meta + (kb & ~1), idesc | (uint32_t)(kb & 1), (it | kb) != 0);
          }
        } else {
#pragma unroll
          for (int kb = 0; kb < 8; ++kb) {                                   // K = 16 each: 32 bytes inside a 128-byte row
            const uint64_t ad = ptx::smem_desc(a_s + (kb >> 2) * 16384 + (kb & 3) * 32, 16, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + (kb >> 2) * (N_TILE * 128) + (kb & 3) * 32, 16, 1024, 2);
            ptx::mma_dense(tmem_base, ad, bd, idesc, (it | kb) != 0);
          }
        }
        ptx::tc_commit(empty_bar(s));
      }
      if (ok) ptx::tc_commit(tmem_full_bar);
    }
  } else if (warp < 2 + EPI_WARPS) {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                               // TMEM lane quadrant this warp may read
    bool ok = true;
    if (num_kt > 0) ok = ptx::mbar_wait_bounded(tmem_full_bar, 0, abort_flag, WAIT_BUDGET);
    if (!ok) *abort_flag = 1;
    ptx::tc_fence_after();
    const int eg = (warp - 2) >> 2;                      // EPI_WARPS / 4 groups of four warps take chunks in turn
    ok = ptx::named_bar_and(1 + eg, 128, ok);            // the four warps of a group go on or give up together
    if (ok) {
      if constexpr (CONV) {
        uint16_t* outp = reinterpret_cast<uint16_t*>(p.out);
        drain_chunks<32>(tmem_base + ((uint32_t)(32 * q) << 16), eg, EPI_GROUPS, N_TILE / 32, num_kt <= 0, 0u,
                         staging + eg * (C::EPI_NT * 8192), 1 + eg, q, lane, p.Mdim - m0, [&](int c, int t) -> uint16_t* {
          // token 32c + t of the box: pixel (cw0 + ., ch0 + .) of image cn0 + .
          const int rr = 32 * c + t;
          const int w = cw0 + (rr & (p.conv.wb - 1));
          const int h = ch0 + ((rr >> p.conv.lg_wb) & (p.conv.hb - 1));
          const int n = cn0 + (rr >> (p.conv.lg_wb + p.conv.lg_hb));
          if (w >= p.conv.W || h >= p.conv.H || n >= p.conv.NB) return nullptr;
          return outp + conv_out_pixel(p.conv, n, h, w) * p.Mdim + m0;
        });
      } else {
        uint32_t u = 0;
        if (!drain_chunks_tma<32, C::EPI_NT>(tmem_base + ((uint32_t)(32 * q) << 16), eg, EPI_GROUPS, N_TILE / 32, num_kt <= 0, 0u,
                                             staging + eg * (C::EPI_NT * 8192), epi_bars_of<C::EPI_NT>(bar_base, eg), u, q, lane,
                                             abort_flag))
          *abort_flag = 1;
      }
    }
  } else if (!CONV) {
    // ------------------------------ store threads: one per epilogue group ------------------------------
    if (ptx::elect_one()) {
      const int g = warp - 2 - EPI_WARPS;
      uint32_t u = 0;
      if (!store_chunks<32, C::EPI_NT>(&tmapD, g, EPI_GROUPS, N_TILE / 32, staging + g * (C::EPI_NT * 8192),
                                       epi_bars_of<C::EPI_NT>(bar_base, g), u, m0, n0, p.Mdim, p.Ndim, abort_flag))
        *abort_flag = 1;
      store_finish();
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


// ------------------------------------------------------------------------------------------
// Persistent CTA-pair 2:4 product.  One pair per two SMs walks 256 x N output tiles in raster
// order.  With N <= 224 (a multiple of 32) tensor memory holds TWO accumulators (columns 0.. and 256..)
// plus the four metadata columns (496..499), so the epilogue of one tile overlaps the main loop of the
// next; N = 256 leaves room for one accumulator only (metadata at 256..259) and is used when the
// tile count would otherwise round up to an extra pass over the SMs (the host picks N).  The TMA
// producer runs ahead across tile boundaries; two groups of four epilogue warps drain an accumulator
// in chunks of 32 columns, taking chunks in turn, and a store warp per group sends the staged chunks
// off as tensor stores (see drain_chunks_tma / store_chunks).
// ------------------------------------------------------------------------------------------


template <int STAGES, bool SPARSE = true>
struct PairPCfg {
  static constexpr int A_BYTES = SPARSE ? 16384 : 32768;   // 128 rows x 64 compressed bf16, or x 128 dense (two boxes)
  static constexpr int B_MAX = 32768;                      // up to 128 rows x 128 bf16 (two 64-wide boxes)
  static constexpr int E_BYTES = SPARSE ? 2048 : 0;
  static constexpr int STAGE_BYTES = A_BYTES + B_MAX + E_BYTES;        // 50 KB / 64 KB (the B part is N / 2 rows)
  static constexpr int EPI_NT = SPARSE ? 3 : 2;            // staging tiles ([32 tokens][128 rows] bf16) per group of four epilogue warps
  static constexpr int STAGING_BYTES = epi_staging_bytes(EPI_NT);
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 + 256;
};

// SPARSE = false: the same kernel on a dense bf16 A operand (masked weights of a pattern the 2:4 format cannot
// hold): a 256 x 128 A tile per stage as two 64-wide boxes per CTA, eight K = 16 MMAs, no metadata, and two
// accumulators at every N (tmapE is not used).
template <int STAGES, bool CONV, bool SPARSE = true>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PAIR_THREADS, 1)
spmm_pair_persistent_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                            const __grid_constant__ CUtensorMap tmapE, const __grid_constant__ CUtensorMap tmapD,
                            const GemmParams p) {
  static_assert(SPARSE || !CONV, "the implicit convolution runs on 2:4 operands only");
  pdl_launch_dependents();
  using C = PairPCfg<STAGES, SPARSE>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t staging = base + STAGES * C::STAGE_BYTES;
  uint8_t* staging_ptr = base_ptr + STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = staging + C::STAGING_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tmem_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tmem_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(staging_ptr + C::STAGING_BYTES + 8 * (2 * STAGES + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n;
  const int num_kt = (p.Kdim + 127) / 128;
  const int SP_N = p.n_tile;                              // output columns (tokens) per tile
  const uint32_t nbuf = (!SPARSE || SP_N <= 240) ? 2u : 1u;   // accumulators in tensor memory
  const uint32_t b_box = (uint32_t)(SP_N / 2) * 128u;     // bytes of one 64-wide box of this CTA's B rows
  const uint32_t stage_tx = C::A_BYTES + 2u * b_box + C::E_BYTES;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(tmem_full_bar(b), 1);
      ptx::mbar_init(tmem_empty_bar(b), 2 * EPI_WARPS);   // the epilogue warps of both CTAs of the pair
    }
    epi_bars_init<C::EPI_NT>(bar_base);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    ptx::prefetch_tmap(&tmapE);
    if (!CONV) ptx::prefetch_tmap(&tmapD);
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
  const uint32_t tmem_meta = tmem_base + (nbuf == 2u ? 496u : 256u);

  if (warp == 0) {
    if (ptx::elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        int tile_m, tile_n;
        raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
        const int mt128 = 2 * tile_m + (int)rank;
        const int m0 = mt128 * 128, nrow = tile_n * SP_N + (SP_N / 2) * (int)rank;
        for (int kt = 0; kt < num_kt; ++kt, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + C::A_BYTES;
          const uint32_t bar = ptx::mapa(full_bar(s), 0);
          if (rank == 0) ptx::mbar_expect_tx(full_bar(s), 2 * stage_tx);
          if (CONV) {
            // this CTA's SP_N / 2 tokens are pixel box 2 * tile_n + rank
            int cw0, ch0, cn0;
            conv_box_origin(p.conv, 2 * tile_n + (int)rank, cw0, ch0, cn0);
            int a_col = kt * 64, a_row = m0, meta_row = mt128, meta_kt = kt;
            if (p.conv.mode == 2) {
              const int tap = kt / p.conv.kt_per_tap;
              meta_kt = kt - tap * p.conv.kt_per_tap;
              a_col = meta_kt * 64;
              a_row = p.conv.tap_id[tap] * p.conv.rows_per_tap + m0;
              meta_row = a_row >> 7;
            }
            ptx::tma_load_2d_pair(a_s, &tmapA, a_col, a_row, bar);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              int c0, dw, dh;
              bool valid;
              conv_k_coords(p.conv, kt, q, p.Kdim, c0, dw, dh, valid);
              ptx::tma_load_4d_pair(b_s + q * b_box, &tmapB, valid ? c0 : 0, p.conv.stride * cw0 + dw, p.conv.stride * ch0 + dh, valid ? cn0 : p.conv.NB, bar);
            }
            ptx::tma_load_2d_pair(b_s + C::B_MAX, &tmapE, 0, 2 * (meta_row * p.tiles_k_meta + meta_kt), bar);
            continue;
          }
          if (SPARSE) {
            ptx::tma_load_2d_pair(a_s, &tmapA, kt * 64, m0, bar);
          } else {
            ptx::tma_load_2d_pair(a_s, &tmapA, kt * 128, m0, bar);
            ptx::tma_load_2d_pair(a_s + 16384, &tmapA, kt * 128 + 64, m0, bar);
          }
          ptx::tma_load_2d_pair(b_s, &tmapB, kt * 128, nrow, bar);
          ptx::tma_load_2d_pair(b_s + b_box, &tmapB, kt * 128 + 64, nrow, bar);
          if (SPARSE) ptx::tma_load_2d_pair(b_s + C::B_MAX, &tmapE, 0, 2 * (mt128 * p.tiles_k_meta + kt), bar);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && ptx::elect_one()) {
      const uint32_t idesc = ptx::idesc_bf16(256, SP_N, false, false, SPARSE);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++tcount) {
        const uint32_t buf = tcount % nbuf;
        // this accumulator must have been drained by both CTAs' epilogues
        if (!ptx::mbar_wait_bounded(tmem_empty_bar(buf), ((tcount / nbuf) & 1u) ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        ptx::tc_fence_after();
        const uint32_t acc = tmem_base + 256u * buf;
        for (int kt = 0; kt < num_kt; ++kt, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + C::A_BYTES;
          if constexpr (SPARSE) {
            ptx::tmem_cp_128x128b_pair(tmem_meta, ptx::smem_desc(b_s + C::B_MAX, 0, 128, 0));
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
              const uint64_t ad = ptx::smem_desc(a_s + kb * 32, 16, 1024, 2);
              const uint64_t bd = ptx::smem_desc(b_s + (kb >> 1) * b_box + (kb & 1) * 64, 16, 1024, 2);
              ptx::mma_sparse_pair(acc, ad, bd, tmem_meta + (kb & ~1), idesc | (uint32_t)(kb & 1), (kt | kb) != 0);
            }
          } else {
#pragma unroll
            for (int kb = 0; kb < 8; ++kb) {                                 // K = 16 each: 32 bytes inside a 128-byte row
              const uint64_t ad = ptx::smem_desc(a_s + (kb >> 2) * 16384 + (kb & 3) * 32, 16, 1024, 2);
              const uint64_t bd = ptx::smem_desc(b_s + (kb >> 2) * b_box + (kb & 3) * 32, 16, 1024, 2);
              ptx::mma_dense_pair(acc, ad, bd, idesc, (kt | kb) != 0);
            }
          }
          ptx::tc_commit_pair(empty_bar(s), 3);
        }
        if (ok) ptx::tc_commit_pair(tmem_full_bar(buf), 3);
      }
    }
  } else if (warp < 2 + EPI_WARPS) {
    // Each epilogue warp reads 32 accumulator rows (its TMEM lane quadrant); the four warps of a group share
    // the group's staging tiles.
    const int q = warp & 3;
    const int eg = (warp - 2) >> 2;                        // EPI_GROUPS groups of four warps take chunks in turn
    const uint32_t stg = staging + eg * (C::EPI_NT * 8192);
    const uint32_t ebars = epi_bars_of<C::EPI_NT>(bar_base, eg);
    uint16_t* outp = reinterpret_cast<uint16_t*>(p.out);
    uint32_t tcount = 0, u = 0;
    for (int tile = cluster_id; tile < num_tiles; tile += num_clusters, ++tcount) {
      int tile_m, tile_n;
      raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
      const int m0 = (2 * tile_m + (int)rank) * 128, n0 = tile_n * SP_N;
      const uint32_t buf = tcount % nbuf;
      bool ok = ptx::mbar_wait_bounded(tmem_full_bar(buf), (tcount / nbuf) & 1u, abort_flag, WAIT_BUDGET);
      ok = ptx::named_bar_and(1 + eg, 128, ok);            // the four warps of a group go on or give up together
      if (!ok) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
      const uint32_t acc = tmem_base + 256u * buf + ((uint32_t)(32 * q) << 16);
      const uint32_t release_bar = ptx::mapa(tmem_empty_bar(buf), 0);
      const int nchunks = SP_N / 32;                        // the hosts pick multiples of 32
      if (CONV) {
        // accumulator columns [0, SP_N/2) are the pixels of box 2*tile_n, the rest those of box 2*tile_n + 1
        drain_chunks<32>(acc, eg, EPI_GROUPS, nchunks, false, release_bar, stg, 1 + eg, q, lane, p.Mdim - m0,
                         [&](int c, int t) -> uint16_t* {
          const int half = (32 * c) / (SP_N / 2);
          const int rr = 32 * c - half * (SP_N / 2) + t;
          int cw0, ch0, cn0;
          conv_box_origin(p.conv, 2 * tile_n + half, cw0, ch0, cn0);
          const int w = cw0 + (rr & (p.conv.wb - 1));
          const int h = ch0 + ((rr >> p.conv.lg_wb) & (p.conv.hb - 1));
          const int n = cn0 + (rr >> (p.conv.lg_wb + p.conv.lg_hb));
          if (w >= p.conv.W || h >= p.conv.H || n >= p.conv.NB) return nullptr;
          return outp + conv_out_pixel(p.conv, n, h, w) * p.Mdim + m0;
        });
      } else if (!drain_chunks_tma<32, C::EPI_NT>(acc, eg, EPI_GROUPS, nchunks, false, release_bar, stg, ebars, u, q, lane,
                                                  abort_flag)) {
        *abort_flag = 1;
        break;
      }
    }
  } else if (!CONV) {
    // store threads, one per epilogue group: the same walk over tiles and chunks as the group's draining warps
    if (ptx::elect_one()) {
      const int g = warp - 2 - EPI_WARPS;
      const uint32_t stg = staging + g * (C::EPI_NT * 8192);
      const uint32_t ebars = epi_bars_of<C::EPI_NT>(bar_base, g);
      uint32_t u = 0;
      for (int tile = cluster_id; tile < num_tiles; tile += num_clusters) {
        int tile_m, tile_n;
        raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
        const int m0 = (2 * tile_m + (int)rank) * 128, n0 = tile_n * SP_N;
        if (!store_chunks<32, C::EPI_NT>(&tmapD, g, EPI_GROUPS, SP_N / 32, stg, ebars, u, m0, n0, p.Mdim, p.Ndim, abort_flag)) {
          *abort_flag = 1;
          break;
        }
      }
      store_finish();
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
// CTA-pair 2:4 product, two row tiles per token tile.  The kernel above streams, per 128-deep k
// tile and CTA, 16 KB of compressed weights + up to 32 KB of activations + 2 KB of metadata for
// 512 tensor-pipe clocks -- about 1.5 x the bytes per clock of the dense kernel, and measurement
// puts it at the L2 -> shared-memory feed rate (tensor pipe 79 % busy, L2 at 60-70 %).  Here a pair
// owns 512 x N outputs: TWO 256-row MMA tiles that share the activation tile in shared memory, so
// a stage carries 2 x 16 KB + <= 28 KB + 2 x 2 KB for twice the tensor-pipe work (a third fewer
// bytes per clock).  Both accumulators (tensor-memory columns 0.. and 256.., N <= 224) belong to
// the same token tile and tensor memory has no room for a second pair, so the epilogue cannot overlap a whole
// main loop; the two groups of four epilogue warps per CTA drain accumulator 0 first, then accumulator 1, and the
// MMA thread starts the next tile's row tile 0 on the stages already loaded while accumulator 1 is still being
// drained (about half of the drain is hidden).  Metadata: columns 496..499 and 500..503.
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-9 epilogue.
// ------------------------------------------------------------------------------------------
constexpr int GEMM2M_THREADS = PAIR_THREADS;

template <int STAGES>
struct Pair2MCfg {
  static constexpr int A_BYTES = 16384;                    // per row tile: 128 rows x 64 compressed bf16
  static constexpr int B_MAX = 28672;                      // 112 rows x 128 bf16 (two 64-wide boxes), N <= 224
  static constexpr int E_BYTES = 2048;
  static constexpr int STAGE_BYTES = 2 * A_BYTES + B_MAX + 2 * E_BYTES;      // 64 KB
  static constexpr int EPI_NT = 2;                         // staging tiles per epilogue group: 8 KB each, and 3 x 64 KB of stages leave room for four
  static constexpr int STAGING_BYTES = epi_staging_bytes(EPI_NT);
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 + 256;
};

template <int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM2M_THREADS, 1)
spmm_pair2m_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                   const __grid_constant__ CUtensorMap tmapE, const __grid_constant__ CUtensorMap tmapD,
                   const GemmParams p) {
  pdl_launch_dependents();
  using C = Pair2MCfg<STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t staging = base + STAGES * C::STAGE_BYTES;
  uint8_t* staging_ptr = base_ptr + STAGES * C::STAGE_BYTES;
  const uint32_t bar_base = staging + C::STAGING_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bar_base + 8u * (2 * STAGES);
  const uint32_t tmem_empty_bar0 = bar_base + 8u * (2 * STAGES + 1);   // accumulator 0 drained
  const uint32_t tmem_empty_bar1 = bar_base + 8u * (2 * STAGES + 2);   // accumulator 1 drained
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(staging_ptr + C::STAGING_BYTES + 8 * (2 * STAGES + 3));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = ptx::cluster_ctarank();
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int num_tiles = p.tiles_m * p.tiles_n;            // tiles_m counts 512-row tiles
  const int num_kt = (p.Kdim + 127) / 128;
  const int SP_N = p.n_tile;                              // tokens per tile, multiple of 32, <= 224
  const uint32_t b_box = (uint32_t)(SP_N / 2) * 128u;     // bytes of one 64-wide box of this CTA's activation rows
  const uint32_t stage_tx = 2u * C::A_BYTES + 2u * b_box + 2u * C::E_BYTES;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(tmem_full_bar, 1);
    ptx::mbar_init(tmem_empty_bar0, 2 * EPI_WARPS);       // the epilogue warps of both CTAs of the pair
    ptx::mbar_init(tmem_empty_bar1, 2 * EPI_WARPS);
    epi_bars_init<C::EPI_NT>(bar_base);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    ptx::prefetch_tmap(&tmapE);
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
  const uint32_t tmem_meta = tmem_base + 496u;            // + 4 * row tile

  // 128-row block of row tile mt (0 / 1) of this CTA inside 512-row tile tile_m
  auto mt128_of = [&](int tile_m, int mt) { return 4 * tile_m + 2 * mt + (int)rank; };

  if (warp == 0) {
    if (ptx::elect_one()) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        int tile_m, tile_n;
        raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
        const int nrow = tile_n * SP_N + (SP_N / 2) * (int)rank;
        for (int kt = 0; kt < num_kt; ++kt, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + 2 * C::A_BYTES;
          const uint32_t e_s = b_s + C::B_MAX;
          const uint32_t bar = ptx::mapa(full_bar(s), 0);
          if (rank == 0) ptx::mbar_expect_tx(full_bar(s), 2 * stage_tx);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            const int mt128 = mt128_of(tile_m, mt);
            ptx::tma_load_2d_pair(a_s + mt * C::A_BYTES, &tmapA, kt * 64, mt128 * 128, bar);
            ptx::tma_load_2d_pair(e_s + mt * C::E_BYTES, &tmapE, 0, 2 * (mt128 * p.tiles_k_meta + kt), bar);
          }
          ptx::tma_load_2d_pair(b_s, &tmapB, kt * 128, nrow, bar);
          ptx::tma_load_2d_pair(b_s + b_box, &tmapB, kt * 128 + 64, nrow, bar);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && ptx::elect_one()) {
      const uint32_t idesc = ptx::idesc_bf16(256, SP_N, false, false, true);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      // the MMAs of row tile mt (0 / 1) on the stage that holds k tile number `it`
      auto issue = [&](uint32_t it_, int kt, int mt) {
        const uint32_t a_s = base + (it_ % STAGES) * C::STAGE_BYTES;
        const uint32_t b_s = a_s + 2 * C::A_BYTES;
        const uint32_t e_s = b_s + C::B_MAX;
        ptx::tmem_cp_128x128b_pair(tmem_meta + 4u * mt, ptx::smem_desc(e_s + mt * C::E_BYTES, 0, 128, 0));
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
          const uint64_t ad = ptx::smem_desc(a_s + mt * C::A_BYTES + kb * 32, 16, 1024, 2);
          const uint64_t bd = ptx::smem_desc(b_s + (kb >> 1) * b_box + (kb & 1) * 64, 16, 1024, 2);
          ptx::mma_sparse_pair(tmem_base + 256u * mt, ad, bd, tmem_meta + 4u * mt + (kb & ~1), idesc | (uint32_t)(kb & 1),
                               (kt | kb) != 0);
        }
      };
      auto wait_full = [&](uint32_t it_) {
        if (!ptx::mbar_wait_bounded(full_bar(it_ % STAGES), (it_ / STAGES) & 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; }
        ptx::tc_fence_after();
        return ok;
      };
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++tcount) {
        // The epilogue drains accumulator 0 first (all sixteen warps of the pair), then accumulator 1.  As soon as
        // accumulator 0 is free, row tile 0 runs ahead over the stages that are already loaded; row tile 1 follows
        // on the same stages once its accumulator is free, and only then are those stages handed back.
        const uint32_t eph = (tcount & 1u) ^ 1u;
        if (!ptx::mbar_wait_bounded(tmem_empty_bar0, eph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        ptx::tc_fence_after();
        const int ahead = num_kt < STAGES ? num_kt : STAGES;
        for (int kt = 0; kt < ahead && ok; ++kt)
          if (wait_full(it + kt)) issue(it + kt, kt, 0);
        if (!ok) break;
        if (!ptx::mbar_wait_bounded(tmem_empty_bar1, eph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
        ptx::tc_fence_after();
        for (int kt = 0; kt < ahead; ++kt) {
          issue(it + kt, kt, 1);
          ptx::tc_commit_pair(empty_bar((it + kt) % STAGES), 3);
        }
        it += ahead;
        for (int kt = ahead; kt < num_kt && ok; ++kt, ++it) {
          if (!wait_full(it)) break;
          issue(it, kt, 0);
          issue(it, kt, 1);
          ptx::tc_commit_pair(empty_bar(it % STAGES), 3);
        }
        if (ok) ptx::tc_commit_pair(tmem_full_bar, 3);
      }
    }
  } else if (warp < 2 + EPI_WARPS) {
    // two groups of four epilogue warps (one warp per tensor-memory lane quadrant); both groups drain accumulator 0
    // first, taking alternate 32-token chunks, then accumulator 1: accumulator 0 is free again at half time, which
    // is what lets the next tile's first MMAs start under the second half of the drain
    const int q = warp & 3;
    const int g = (warp - 2) >> 2;
    const uint32_t stg = staging + g * (C::EPI_NT * 8192);
    const uint32_t ebars = epi_bars_of<C::EPI_NT>(bar_base, g);
    uint32_t u = 0;
    const uint32_t release0 = ptx::mapa(tmem_empty_bar0, 0), release1 = ptx::mapa(tmem_empty_bar1, 0);
    uint32_t tcount = 0;
    for (int tile = cluster_id; tile < num_tiles; tile += num_clusters, ++tcount) {
      bool ok = ptx::mbar_wait_bounded(tmem_full_bar, tcount & 1u, abort_flag, WAIT_BUDGET);
      ok = ptx::named_bar_and(1 + g, 128, ok);             // the four warps of a group go on or give up together
      if (!ok) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
#pragma unroll 1
      for (int mt = 0; mt < 2; ++mt) {
        const uint32_t acc = tmem_base + 256u * mt + ((uint32_t)(32 * q) << 16);
        if (!drain_chunks_tma<32, C::EPI_NT>(acc, (g ^ mt) & 1, 2, SP_N / 32, false, mt ? release1 : release0, stg, ebars, u, q,
                                             lane, abort_flag))
          *abort_flag = 1;
      }
      if (*abort_flag) break;
    }
  } else {
    // store threads, one per epilogue group: the same walk over tiles, row tiles and chunks as the group's draining warps
    if (ptx::elect_one()) {
      const int g = warp - 2 - EPI_WARPS;
      const uint32_t stg = staging + g * (C::EPI_NT * 8192);
      const uint32_t ebars = epi_bars_of<C::EPI_NT>(bar_base, g);
      uint32_t u = 0;
      bool ok = true;
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters) {
        int tile_m, tile_n;
        raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
        for (int mt = 0; mt < 2 && ok; ++mt)
          ok = store_chunks<32, C::EPI_NT>(&tmapD, (g ^ mt) & 1, 2, SP_N / 32, stg, ebars, u, mt128_of(tile_m, mt) * 128, tile_n * SP_N,
                                           p.Mdim, p.Ndim, abort_flag);
      }
      if (!ok) *abort_flag = 1;
      store_finish();
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

template <int N_TILE, int STAGES, bool SPARSE = true>
int run_single(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
               uint16_t* out, int32_t* status_word, cudaStream_t s) {
  using C = Cfg<N_TILE, STAGES, SPARSE>;
  CUtensorMap ta, tb, td;
  int rc;
  if ((rc = make_tmap(&ta, vals, SPARSE ? (uint64_t)Kdim / 2 : (uint64_t)Kdim, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, N_TILE)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&td, out, (uint64_t)Mdim, (uint64_t)Ndim, 32)) != BIMASK_OK) return rc;   // result: 32 tokens x 64 rows per store
  auto kern = spmm_single_kernel<N_TILE, STAGES, SPARSE, false>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv.mode = 0;
  p.hw_meta = reinterpret_cast<const uint8_t*>(hw_meta);
  p.tiles_k_meta = (Kdim + 127) / 128;
  p.Mdim = Mdim; p.Ndim = Ndim; p.Kdim = Kdim;
  p.k_tiles_per_split = (Kdim + 127) / 128;
  p.out = out;
  p.status_word = status_word;
  p.tiles_m = (Mdim + 127) / 128;
  p.tiles_n = (Ndim + N_TILE - 1) / N_TILE;
  p.raster_group = 16;
  dim3 grid(p.tiles_m * p.tiles_n, 1, 1);
  BIMASK_CUDA_OK(launch_pdl(kern, grid, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, td, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// Output-tile width of the CTA-pair 2:4 product.  Cost model in SM clocks, fitted to measurements: per 128-deep k
// tile a CTA takes in 18 KB of compressed weights and metadata plus 128 N bytes of activations at about 64 bytes per
// clock (short reductions and narrow tiles are bound by that, not by the 2 N clocks of the MMAs); the epilogue (two
// groups of four draining warps, a store warp each) takes about 430 clocks per 32-column chunk and group; with
// N <= 224 the two overlap (two accumulators), with N = 256 they add up; the kernel's time is the number of passes
// over the clusters times the tile time.
int choose_sparse_n(int pair_tiles_m, int Ndim, int k_tiles, int clusters) {
  int best_n = 256;
  double best = 1e30;
  for (int n = 256; n >= 96; n -= 32) {                     // multiples of 32 only: 16-column chunks drain at 570 clocks each
    const long long tiles = (long long)pair_tiles_m * ((Ndim + n - 1) / n);
    const long long rounds = (tiles + clusters - 1) / clusters;
    const double feed = (18432.0 + 128.0 * n) / 64.0;
    const double mainloop = (double)k_tiles * (2.0 * n > feed ? 2.0 * n : feed);
    const double epilogue = ((n / 32 + 1) / 2) * 430.0;
    const double tile = n == 256 ? mainloop + epilogue : (mainloop > epilogue ? mainloop : epilogue);
    const double cost = (double)rounds * tile * (1.0 + 0.001 * (256 - n));
    if (cost < best) { best = cost; best_n = n; }
  }
  return best_n;
}

int run_sparse_pair_persistent(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim,
                               int Kdim, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  constexpr int STAGES = 3;
  using C = PairPCfg<STAGES>;
  CUtensorMap ta, tb, te, td;
  int rc;
  const int tiles_m = (Mdim + 127) / 128, tiles_k = (Kdim + 127) / 128;
  const int sms = sm_count();
  const int n_tile = choose_sparse_n((tiles_m + 1) / 2, Ndim, tiles_k, sms / 2);
  if ((rc = make_tmap(&ta, vals, (uint64_t)Kdim / 2, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, n_tile / 2)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_meta(&te, hw_meta, (uint64_t)tiles_m * tiles_k)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&td, out, (uint64_t)Mdim, (uint64_t)Ndim, 32)) != BIMASK_OK) return rc;   // one chunk of the drain: 32 tokens x 64 rows per store
  auto kern = spmm_pair_persistent_kernel<STAGES, false>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv.mode = 0;
  p.hw_meta = reinterpret_cast<const uint8_t*>(hw_meta);
  p.tiles_k_meta = tiles_k;
  p.Mdim = Mdim; p.Ndim = Ndim; p.Kdim = Kdim;
  p.k_tiles_per_split = tiles_k;
  p.out = out;
  p.status_word = status_word;
  p.n_tile = n_tile;
  p.tiles_m = (tiles_m + 1) / 2;
  p.tiles_n = (Ndim + n_tile - 1) / n_tile;
  p.raster_group = 8;
  const int total = p.tiles_m * p.tiles_n;
  const int clusters = total < sms / 2 ? total : sms / 2;
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, te, td, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// Token-tile width of the two-row-tile kernel: per 128-deep k tile a pair issues eight MMAs of N / 2
// clocks; the epilogue (not overlapped) costs about 2500 clocks per tile.
int choose_sparse_n_2m(int tiles_m512, int Ndim, int k_tiles, int clusters) {
  int best_n = 224;
  double best = 1e30;
  for (int n = 224; n >= 160; n -= 32) {
    const long long tiles = (long long)tiles_m512 * ((Ndim + n - 1) / n);
    const long long rounds = (tiles + clusters - 1) / clusters;
    const double cost = (double)rounds * ((double)k_tiles * 4.0 * n + 2500.0) * (1.0 + 0.003 * (224 - n));
    if (cost < best) { best = cost; best_n = n; }
  }
  return best_n;
}

int run_sparse_pair2m(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
                      uint16_t* out, int32_t* status_word, cudaStream_t s) {
  constexpr int STAGES = 3;
  using C = Pair2MCfg<STAGES>;
  CUtensorMap ta, tb, te, td;
  int rc;
  const int tiles_m = (Mdim + 127) / 128, tiles_k = (Kdim + 127) / 128;
  const int sms = sm_count();
  const int tiles_m512 = (tiles_m + 3) / 4;
  const int n_tile = choose_sparse_n_2m(tiles_m512, Ndim, tiles_k, sms / 2);
  if ((rc = make_tmap(&ta, vals, (uint64_t)Kdim / 2, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, n_tile / 2)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_meta(&te, hw_meta, (uint64_t)tiles_m * tiles_k)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&td, out, (uint64_t)Mdim, (uint64_t)Ndim, 32)) != BIMASK_OK) return rc;
  auto kern = spmm_pair2m_kernel<STAGES>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv.mode = 0;
  p.hw_meta = reinterpret_cast<const uint8_t*>(hw_meta);
  p.tiles_k_meta = tiles_k;
  p.Mdim = Mdim; p.Ndim = Ndim; p.Kdim = Kdim;
  p.k_tiles_per_split = tiles_k;
  p.out = out;
  p.status_word = status_word;
  p.n_tile = n_tile;
  p.tiles_m = tiles_m512;
  p.tiles_n = (Ndim + n_tile - 1) / n_tile;
  // eight 512-row tiles of one token tile run side by side: measured against 4 on the config-5 products, DRAM reads
  // fall by 40 % (610 -> 363 MB, 614 -> 358 MB) and the products take 3 % less time; 2 and 32 are worse on both counts
  p.raster_group = 8;
  const int total = p.tiles_m * p.tiles_n;
  const int clusters = total < sms / 2 ? total : sms / 2;
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, GEMM2M_THREADS, C::SMEM_BYTES, s, ta, tb, te, td, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace

int launch_spmm(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
                uint16_t* out, int32_t* status_word, cudaStream_t s) {
  // large operands with a long reduction: two row tiles per token tile (fewer bytes per tensor-pipe clock; its
  // epilogue is not overlapped, which pays off from about 28 k tiles: measured 2 % faster at k = 4096, 8-10 % at
  // k = 16384)
  if (Ndim >= 1024 && Mdim >= 2048 && Kdim >= 4096)
    return run_sparse_pair2m(vals, hw_meta, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  if (Ndim > 128 && Mdim > 128) return run_sparse_pair_persistent(vals, hw_meta, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  if (Ndim > 128) return run_single<256, 2>(vals, hw_meta, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  return run_single<128, 3>(vals, hw_meta, Bop, Mdim, Ndim, Kdim, out, status_word, s);
}

namespace {

template <int N_TILE, int STAGES>
int run_conv_single(const uint16_t* vals, int a_rows, int a_kdim, const void* hw_meta, const uint16_t* tok, int in_h, int in_w, ConvGeom g,
                    int Mdim, int Kdim, int tiles_k_meta, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  using C = Cfg<N_TILE, STAGES, true>;
  conv_boxes(g, N_TILE);
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap(&ta, vals, (uint64_t)a_kdim / 2, (uint64_t)a_rows, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_nhwc_load(&tb, tok, g.CB, in_w, in_h, g.NB, g.wb, g.hb, g.nb, g.stride)) != BIMASK_OK) return rc;
  auto kern = spmm_single_kernel<N_TILE, STAGES, true, true>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv = g;
  p.hw_meta = reinterpret_cast<const uint8_t*>(hw_meta);
  p.tiles_k_meta = tiles_k_meta;
  p.Mdim = Mdim; p.Ndim = g.NB * g.H * g.W; p.Kdim = Kdim;
  p.k_tiles_per_split = (Kdim + 127) / 128;
  p.out = out;
  p.status_word = status_word;
  p.tiles_m = (Mdim + 127) / 128;
  p.tiles_n = g.tiles_w * g.tiles_h * ((g.NB + g.nb - 1) / g.nb);
  p.raster_group = 16;
  p.n_tile = N_TILE;
  dim3 grid(p.tiles_m * p.tiles_n, 1, 1);
  BIMASK_CUDA_OK(launch_pdl(kern, grid, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, ta /* result map: not used by the convolution */, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int run_conv_pair(const uint16_t* vals, int a_rows, int a_kdim, const void* hw_meta, const uint16_t* tok, int in_h, int in_w, ConvGeom g,
                  int Mdim, int Kdim, int tiles_k_meta, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  constexpr int STAGES = 3;
  using C = PairPCfg<STAGES>;
  const int n_tile = 128;                                // two boxes of 64 pixels; two accumulators in tensor memory
  conv_boxes(g, n_tile / 2);
  CUtensorMap ta, tb, te;
  int rc;
  const int a_tiles_m = (a_rows + 127) / 128;
  const int sms = sm_count();
  if ((rc = make_tmap(&ta, vals, (uint64_t)a_kdim / 2, (uint64_t)a_rows, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_nhwc_load(&tb, tok, g.CB, in_w, in_h, g.NB, g.wb, g.hb, g.nb, g.stride)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_meta(&te, hw_meta, (uint64_t)a_tiles_m * tiles_k_meta)) != BIMASK_OK) return rc;
  auto kern = spmm_pair_persistent_kernel<STAGES, true>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv = g;
  p.hw_meta = reinterpret_cast<const uint8_t*>(hw_meta);
  p.tiles_k_meta = tiles_k_meta;
  p.Mdim = Mdim; p.Ndim = g.NB * g.H * g.W; p.Kdim = Kdim;
  p.k_tiles_per_split = (Kdim + 127) / 128;
  p.out = out;
  p.status_word = status_word;
  p.n_tile = n_tile;
  p.tiles_m = ((Mdim + 127) / 128 + 1) / 2;
  const int boxes = g.tiles_w * g.tiles_h * ((g.NB + g.nb - 1) / g.nb);
  p.tiles_n = (boxes + 1) / 2;
  p.raster_group = 8;
  const int total = p.tiles_m * p.tiles_n;
  const int clusters = total < sms / 2 ? total : sms / 2;
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, te, ta /* result map: not used by the convolution */, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace

// 3x3 convolution products without a column matrix (see ConvGeom).
//   forward:        D[i, pixel] = sum_{tap, c} A_f[i, tap*C + c] x[pixel + tap, c];  vals/hw_meta of the I x 9C operand
//   input gradient: D[c, pixel] = sum_{tap, i'} A'[tap*C + c, i'] dyp[pixel - tap, i'];  vals/hw_meta of the 9C x I operand
// out is NHWC with Mdim channels.  Needs C % 64 == 0 (forward); C % 128 == 0 or C == 64 (input gradient).
int launch_spmm_conv(int mode, const uint16_t* vals, const void* hw_meta, const uint16_t* tok, int NB, int H, int W, int C,
                     int I, int stride, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  ConvGeom g{};
  g.mode = mode; g.NB = NB;
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;       // the convolution's output image
  auto run = [&](const ConvGeom& gg, int tok_h, int tok_w, int Mdim, int Kdim, int a_rows, int a_kdim, int tiles_k_meta) {
    const long long T = (long long)NB * gg.H * gg.W;
    if (Mdim > 128 && T > 128)
      return run_conv_pair(vals, a_rows, a_kdim, hw_meta, tok, tok_h, tok_w, gg, Mdim, Kdim, tiles_k_meta, out, status_word, s);
    if (T > 128)
      return run_conv_single<256, 2>(vals, a_rows, a_kdim, hw_meta, tok, tok_h, tok_w, gg, Mdim, Kdim, tiles_k_meta, out, status_word, s);
    return run_conv_single<128, 3>(vals, a_rows, a_kdim, hw_meta, tok, tok_h, tok_w, gg, Mdim, Kdim, tiles_k_meta, out, status_word, s);
  };
  if (mode == 1) {
    // the tokens are the output pixels; with stride 2 the input tensor map is traversed with stride 2
    g.stride = stride; g.H = Ho; g.W = Wo;
    g.CB = C; g.kt_per_tap = 0; g.rows_per_tap = 0;
    g.out_step = 1; g.out_h0 = 0; g.out_w0 = 0; g.out_H = Ho; g.out_W = Wo;
    return run(g, H, W, I, 9 * C, I, 9 * C, (9 * C + 127) / 128);
  }
  // input gradient: the tokens are pixels of dx (H x W), the token operand is the permuted dy (Ho x Wo), read with unit stride
  g.stride = 1;
  g.CB = I; g.kt_per_tap = (I + 127) / 128; g.rows_per_tap = C;
  g.out_H = H; g.out_W = W;
  if (stride == 1) {
    g.H = H; g.W = W;
    g.out_step = 1; g.out_h0 = 0; g.out_w0 = 0;
    for (int t = 0; t < 9; ++t) { g.tap_id[t] = (signed char)t; g.tap_dh[t] = (signed char)(1 - t / 3); g.tap_dw[t] = (signed char)(1 - t % 3); }
    return run(g, Ho, Wo, C, 9 * g.kt_per_tap * 128, 9 * C, I, g.kt_per_tap);
  }
  BIMASK_REQUIRE(stride == 2, BIMASK_EUNSUPPORTED, "implicit input gradient: stride %d", stride);
  // stride 2: one stride-1 problem per parity class of the input pixels (see ConvGeom)
  for (int ph = 0; ph < 2; ++ph)
    for (int pw = 0; pw < 2; ++pw) {
      ConvGeom gc = g;
      gc.H = (H - ph + 1) / 2; gc.W = (W - pw + 1) / 2;
      if (gc.H <= 0 || gc.W <= 0) continue;
      gc.out_step = 2; gc.out_h0 = ph; gc.out_w0 = pw;
      int nt = 0;
      for (int kh = 0; kh < 3; ++kh)
        for (int kw = 0; kw < 3; ++kw) {
          if (((ph + 1 - kh) & 1) || ((pw + 1 - kw) & 1)) continue;
          gc.tap_id[nt] = (signed char)(kh * 3 + kw);
          gc.tap_dh[nt] = (signed char)((ph + 1 - kh) / 2);
          gc.tap_dw[nt] = (signed char)((pw + 1 - kw) / 2);
          ++nt;
        }
      const int rc = run(gc, Ho, Wo, C, nt * g.kt_per_tap * 128, 9 * C, I, g.kt_per_tap);
      if (rc != BIMASK_OK) return rc;
    }
  return BIMASK_OK;
}

namespace {

// Dense operand, CTA pairs: 256 x N tiles, N the multiple of 32 (at most 256) that wastes the fewest token columns
// among those with the fewest rounds over the pairs.
int run_dense_pair_persistent(const uint16_t* A, const uint16_t* Bop, int Mdim, int Ndim, int Kdim, uint16_t* out,
                              int32_t* status_word, cudaStream_t s) {
  constexpr int STAGES = 3;
  using C = PairPCfg<STAGES, false>;
  CUtensorMap ta, tb, td;
  int rc;
  const int tiles_m = (Mdim + 127) / 128, tiles_k = (Kdim + 127) / 128;
  const int sms = sm_count();
  int n_tile = 256;
  double best = 1e30;
  for (int n = 256; n >= 160; n -= 32) {
    const long long tiles = (long long)((tiles_m + 1) / 2) * ((Ndim + n - 1) / n);
    const long long rounds = (tiles + sms / 2 - 1) / (sms / 2);
    const double cost = (double)rounds * n * (1.0 + 0.002 * (256 - n));
    if (cost < best) { best = cost; n_tile = n; }
  }
  if ((rc = make_tmap(&ta, A, (uint64_t)Kdim, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, n_tile / 2)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&td, out, (uint64_t)Mdim, (uint64_t)Ndim, 32)) != BIMASK_OK) return rc;
  auto kern = spmm_pair_persistent_kernel<STAGES, false, false>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv.mode = 0;
  p.hw_meta = nullptr;
  p.tiles_k_meta = tiles_k;
  p.Mdim = Mdim; p.Ndim = Ndim; p.Kdim = Kdim;
  p.k_tiles_per_split = tiles_k;
  p.out = out;
  p.status_word = status_word;
  p.n_tile = n_tile;
  p.tiles_m = (tiles_m + 1) / 2;
  p.tiles_n = (Ndim + n_tile - 1) / n_tile;
  p.raster_group = 8;
  const int total = p.tiles_m * p.tiles_n;
  const int clusters = total < sms / 2 ? total : sms / 2;
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, ta /* no metadata */, td, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace

int launch_dense_nt(const uint16_t* A, const uint16_t* Bop, int Mdim, int Ndim, int Kdim, uint16_t* out,
                    int32_t* status_word, cudaStream_t s) {
  if (Ndim > 128 && Mdim > 128) return run_dense_pair_persistent(A, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  if (Ndim > 128) return run_single<256, 2, false>(A, nullptr, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  return run_single<128, 3, false>(A, nullptr, Bop, Mdim, Ndim, Kdim, out, status_word, s);
}

}  // namespace bimask
