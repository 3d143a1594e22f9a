// The three products of the layer step on the 5th-generation tensor cores:
//   sparse forward    D[i, t] = sum_j A_f[i, j] X[t, j]        (Eq. 3;  A_f 2:4 along j)
//   sparse input grad D[l, t] = sum_k A'[l, k] dYp[t, k]       (Eq. 10; A' 2:4 along permuted k)
//   dense weight grad D[i, j] = sum_t dY[t, i] X[t, j]         (straight-through estimator)
//
// All kernels are warp-specialised: a TMA producer thread fills a ring of shared-memory stages
// (operands in the 128-byte-swizzled layouts the tensor core reads directly), one thread issues
// tcgen05.mma (.sp for the 2:4 operand, whose index metadata is copied shared -> tensor memory
// with tcgen05.cp right before the MMAs that use it), accumulators live in tensor memory, and
// four epilogue warps drain them with tcgen05.ld and store the result.  The large-shape kernels
// (spmm_pair_persistent_kernel, wgrad_pair_kernel) run CTA pairs persistently; spmm_single_kernel
// is the one-CTA-per-tile form for operands of at most 128 rows or at most 128 tokens.
//
// Every wait on an mbarrier carries a cycle budget: when it runs out the kernel writes
// BIMASK_ETIMEOUT to the caller's status word, all roles unwind, tensor memory is released and
// the kernel returns.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include <cuda_bf16.h>
#include <atomic>
#include <mutex>

namespace bimask {

namespace {

constexpr long long WAIT_BUDGET = 4000000000ll;      // ~2 s of SM clocks
constexpr int GEMM_THREADS = 192;                    // warp 0 TMA, warp 1 MMA, warps 2-5 epilogue
// The sparse kernels that drain bf16 results use eight epilogue warps (two groups of four, one warp per
// tensor-memory lane quadrant, taking alternate column chunks): products with a short reduction are bound by
// that drain, not by the tensor pipe.
constexpr int EPI_WARPS = 8;
constexpr int PAIR_THREADS = 64 + 32 * EPI_WARPS;

template <int N_TILE, int STAGES, bool SPARSE = true>
struct Cfg {
  static constexpr int M_TILE = 128;
  static constexpr int K_TILE = 128;                             // logical reduction elements per stage
  static constexpr int A_BYTES = SPARSE ? 16384 : 32768;         // 128 rows x 64 compressed, or x 128 dense, bf16
  static constexpr int B_BYTES = N_TILE * K_TILE * 2;
  static constexpr int E_BYTES = SPARSE ? 2048 : 0;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
  static constexpr int META_COLS = SPARSE ? 4 : 0;
  static constexpr int TMEM_COLS = (N_TILE + META_COLS) <= 128 ? 128 : (N_TILE + META_COLS) <= 256 ? 256 : 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */ +
                                    EPI_WARPS * 2048 /* epilogue staging: one [32 tokens][128 rows] bf16 tile per group of four warps */;
};

// A 3x3 convolution as an implicit GEMM: the token operand is an NHWC tensor and a "tile of
// tokens" is a box of wb x hb pixels of nb images, fetched with one 4-D tensor load per 64
// channels, shifted by the filter tap the k index belongs to (pixels outside the image read 0).
//   mode 1 (forward, Eq. 3):        k = (tap, c);  B = x,   shift (+kw-1, +kh-1)
//   mode 2 (input gradient, Eq. 10): k = (tap, i');  B = dy[:, perm], shift (1-kw, 1-kh); the rows of
//           the 2:4 operand for tap (kh, kw) are (kh*3+kw)*C + c.
struct ConvGeom {
  int mode;                 // 0: plain matrix operand
  int H, W, NB;             // image
  int CB;                   // channels of the token operand (x: C; dy: I)
  int wb, hb, nb;           // pixel box of one load: wb * hb * nb tokens (powers of two)
  int lg_wb, lg_hb;         // their logarithms
  int tiles_w, tiles_h;     // boxes per image
  int kt_per_tap;           // mode 2: 128-wide k tiles per filter tap (I / 128)
  int rows_per_tap;         // mode 2: rows of the 2:4 operand per tap (C)
};

__device__ __forceinline__ void conv_box_origin(const ConvGeom& g, int box, int& w0, int& h0, int& n0) {
  w0 = (box % g.tiles_w) * g.wb;
  const int r = box / g.tiles_w;
  h0 = (r % g.tiles_h) * g.hb;
  n0 = (r / g.tiles_h) * g.nb;
}

// Channel offset and pixel shift of the 64-wide half q of k tile kt; valid = false: past the
// reduction length (the loader then reads a box of zeros).
__device__ __forceinline__ void conv_k_coords(const ConvGeom& g, int kt, int q, int Kdim, int& c0, int& dw, int& dh, bool& valid) {
  if (g.mode == 1) {
    const int j = kt * 128 + 64 * q;
    valid = j < Kdim;
    const int tap = j / g.CB;
    c0 = j - tap * g.CB;
    dh = tap / 3 - 1;
    dw = tap % 3 - 1;
  } else {
    const int tap = kt / g.kt_per_tap;
    c0 = (kt - tap * g.kt_per_tap) * 128 + 64 * q;
    valid = true;
    dh = 1 - tap / 3;
    dw = 1 - tap % 3;
  }
}

struct GemmParams {
  ConvGeom conv;
  const uint8_t* hw_meta;   // sparse only
  int tiles_k_meta;         // number of 128-wide k tiles in the metadata image
  int Mdim, Ndim, Kdim;     // D is Mdim x Ndim, reduction length Kdim (logical)
  int k_tiles_per_split;    // dense split-K: k tiles handled by one blockIdx.z
  int tiles_m, tiles_n;     // output tiles (CTA pairs along M for the pair kernel)
  int raster_group;         // tiles walked along M before advancing along N
  int n_tile;               // pair kernel: output columns per tile (multiple of 16, <= 256)
  void* out;                // sparse: bf16 [Ndim][Mdim];  dense: fp32 [split][Mdim][Ndim]
  int32_t* status_word;
};


// Tile order.  A linear id walks `group` tiles along M before it advances along N, so that the
// CTAs resident at one time cover a near-square patch of the output and both operands are
// re-used out of L2 instead of being streamed from HBM once per wave.
__device__ __forceinline__ void raster(int id, int tiles_m, int tiles_n, int group, int& tm, int& tn) {
  const int per_group = group * tiles_n;
  const int g = id / per_group;
  const int first = g * group;
  const int gsize = min(group, tiles_m - first);
  const int in = id - g * per_group;
  tm = first + in % gsize;
  tn = in / gsize;
}

// Epilogue of the 2:4 products.  The accumulator holds D[row][token] (row = tensor-memory lane), the result is
// stored token-major, so a chunk of W tokens x the CTA's 128 rows is transposed on its way out by a GROUP of four
// warps, one per tensor-memory lane quadrant:
//   tensor memory -> registers in the accumulator-fragment layout (two 16-lane loads per warp) -> bf16 pairs ->
//   stmatrix.trans into the group's staging tile [token][128 rows] (256-byte rows; the 16-byte unit index is
//   XOR-ed with the token index mod 8, so the eight rows of a matrix fall into eight different bank groups) ->
//   named barrier -> each warp reads W/4 whole token rows back and writes them with 16-byte stores, 256 contiguous
//   bytes per token (whole 128-byte lines: half-line writes were bound by the number of write requests).
// The tensor-memory load of the next chunk is issued before the current one is converted and stored.
template <int W>
__device__ __forceinline__ void epi_load(uint32_t taddr, uint32_t (&r)[W], bool zero) {
  if (zero) {
#pragma unroll
    for (int j = 0; j < W; ++j) r[j] = 0u;
  } else if (W == 32) {
    ptx::tmem_ld_16x256b_x4(taddr, &r[0]);                 // lanes 0-15 of the quadrant
    ptx::tmem_ld_16x256b_x4(taddr + (16u << 16), &r[16]);  // lanes 16-31
  } else {
    ptx::tmem_ld_16x256b_x2(taddr, &r[0]);
    ptx::tmem_ld_16x256b_x2(taddr + (16u << 16), &r[W / 2]);
  }
}

__device__ __forceinline__ uint32_t pack_bf16(uint32_t lo, uint32_t hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(lo), __uint_as_float(hi));
  return *reinterpret_cast<const uint32_t*>(&v);
}

// `dst`: this lane's row address for token group 0 (see drain_chunks); token group g is 2048 bytes further.
template <int W>
__device__ __forceinline__ void epi_stage(const uint32_t (&r)[W], uint32_t dst) {
#pragma unroll
  for (int g = 0; g < W / 8; ++g)
    ptx::stmatrix_x4_trans(dst + 2048u * g, pack_bf16(r[4 * g], r[4 * g + 1]), pack_bf16(r[4 * g + 2], r[4 * g + 3]),
                           pack_bf16(r[W / 2 + 4 * g], r[W / 2 + 4 * g + 1]),
                           pack_bf16(r[W / 2 + 4 * g + 2], r[W / 2 + 4 * g + 3]));
}

// Drains chunks c0, c0 + cstep, ... (< nchunks) of one accumulator; called by the four warps of a group with the
// same arguments except `acc` (the warp's lane quadrant q = warp % 4, column of chunk c: W * c).  After its last
// tensor-memory read each warp arrives once on `release_bar` (0: nobody waits for the accumulator).
// row_of(c, t) returns where token t of chunk c starts in the result (the CTA's first row), or nullptr when that
// token lies outside; rows_valid = how many of the CTA's 128 rows exist (a multiple of 32).
// `stg`: the group's staging tile (W * 256 bytes, 1 KB aligned); `bar_id`: its named barrier.
template <int W, typename RowOf>
__device__ __forceinline__ void drain_chunks(uint32_t acc, int c0, int cstep, int nchunks, bool zero, uint32_t release_bar,
                                             uint32_t stg, uint32_t bar_id, int q, int lane, int rows_valid, RowOf&& row_of) {
  auto release = [&]() {
    if (release_bar != 0u) {
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(release_bar);
    }
  };
  if (c0 >= nchunks) { release(); return; }
  // stmatrix: lane 8 i + k addresses token k (of a group of eight) of matrix i = rows 32 q + 8 i .. + 7, i.e. unit
  // 4 q + i of the token's 256-byte row
  const uint32_t dst = stg + (uint32_t)(lane & 7) * 256u + ((((uint32_t)(4 * q) + ((uint32_t)lane >> 3)) ^ ((uint32_t)lane & 7u)) << 4);
  // reading back: this warp owns tokens (W/4) q .. (W/4) q + W/4 - 1; per step lanes 0-15 take one token, lanes 16-31
  // the next, 16 bytes (eight rows) per lane
  const int unit = lane & 15;
  const bool unit_ok = 8 * unit < rows_valid;
  auto emit = [&](const uint32_t (&r)[W], int c) {
    ptx::named_bar_sync(bar_id, 128);                     // the group has read the previous chunk out of the tile
    epi_stage<W>(r, dst);
    ptx::named_bar_sync(bar_id, 128);
#pragma unroll
    for (int i = 0; i < W / 8; ++i) {
      const int t = (W / 4) * q + 2 * i + (lane >> 4);
      const uint4 v = ptx::ld_shared_v4(stg + (uint32_t)t * 256u + (((uint32_t)unit ^ ((uint32_t)t & 7u)) << 4));
      uint16_t* row = row_of(c, t);
      if (row != nullptr && unit_ok) *reinterpret_cast<uint4*>(row + 8 * unit) = v;
    }
  };
  uint32_t ra[W], rb[W];
  epi_load<W>(acc + W * c0, ra, zero);
#pragma unroll 1
  for (int c = c0; c < nchunks; c += 2 * cstep) {
    if (!zero) ptx::tmem_ld_wait();
    const bool more1 = c + cstep < nchunks;
    if (more1) epi_load<W>(acc + W * (c + cstep), rb, zero); else release();
    emit(ra, c);
    if (!more1) break;
    if (!zero) ptx::tmem_ld_wait();
    if (c + 2 * cstep < nchunks) epi_load<W>(acc + W * (c + 2 * cstep), ra, zero); else release();
    emit(rb, c + cstep);
  }
}

// SPARSE = false: the same pipeline on a dense bf16 A operand (masked weights of a pattern the
// 2:4 format cannot hold): 128 x 128 A tile per stage as two 64-wide boxes, eight K = 16 MMAs.
// CONV: the token operand is fetched as shifted pixel boxes (see ConvGeom); N_TILE tokens = one box.
template <int N_TILE, int STAGES, bool SPARSE, bool CONV>
__global__ void __launch_bounds__(PAIR_THREADS, 1)
spmm_single_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                   const GemmParams p) {
  pdl_launch_dependents();
  using C = Cfg<N_TILE, STAGES, SPARSE>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t staging = base + STAGES * C::STAGE_BYTES;      // epilogue staging, 8 KB per group of four warps
  const uint32_t bar_base = staging + EPI_WARPS * 2048;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bar_base + 8u * (2 * STAGES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + EPI_WARPS * 2048 + 8 * (2 * STAGES + 1));
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
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
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
            a_row = tap * p.conv.rows_per_tap + m0;
            meta_row = a_row >> 7;
          }
          ptx::tma_load_2d(a_s, &tmapA, a_col, a_row, full_bar(s));
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            int c0, dw, dh;
            bool valid;
            conv_k_coords(p.conv, kt, q, p.Kdim, c0, dw, dh, valid);
            ptx::tma_load_4d(b_s + q * (N_TILE * 128), &tmapB, valid ? c0 : 0, cw0 + dw, ch0 + dh, valid ? cn0 : p.conv.NB,
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
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                               // TMEM lane quadrant this warp may read
    bool ok = true;
    if (num_kt > 0) ok = ptx::mbar_wait_bounded(tmem_full_bar, 0, abort_flag, WAIT_BUDGET);
    if (!ok) *abort_flag = 1;
    ptx::tc_fence_after();
    const int eg = (warp - 2) >> 2;                      // EPI_WARPS / 4 groups of four warps take chunks in turn
    ok = ptx::named_bar_and(1 + eg, 128, ok);            // the four warps of a group go on or give up together
    if (ok) {
      uint16_t* outp = reinterpret_cast<uint16_t*>(p.out);
      drain_chunks<32>(tmem_base + ((uint32_t)(32 * q) << 16), eg, EPI_WARPS / 4, N_TILE / 32, num_kt <= 0, 0u,
                       staging + eg * 8192, 1 + eg, q, lane, p.Mdim - m0, [&](int c, int t) -> uint16_t* {
        if (CONV) {
          // token 32c + t of the box: pixel (cw0 + ., ch0 + .) of image cn0 + .
          const int rr = 32 * c + t;
          const int w = cw0 + (rr & (p.conv.wb - 1));
          const int h = ch0 + ((rr >> p.conv.lg_wb) & (p.conv.hb - 1));
          const int n = cn0 + (rr >> (p.conv.lg_wb + p.conv.lg_hb));
          if (w >= p.conv.W || h >= p.conv.H || n >= p.conv.NB) return nullptr;
          return outp + ((size_t)(n * p.conv.H + h) * p.conv.W + w) * p.Mdim + m0;
        }
        const int n = n0 + 32 * c + t;
        return n < p.Ndim ? outp + (size_t)n * p.Mdim + m0 : nullptr;
      });
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
// order.  With N <= 240 tensor memory holds TWO accumulators (columns 0.. and 256..) plus the
// four metadata columns (496..499), so the epilogue of one tile overlaps the main loop of the
// next; N = 256 leaves room for one accumulator only (metadata at 256..259) and is used when the
// tile count would otherwise round up to an extra pass over the SMs (the host picks N).  The TMA
// producer runs ahead across tile boundaries; two groups of four epilogue warps drain an accumulator
// in chunks of 32 (16) columns, taking chunks in turn (see drain_chunks).
// ------------------------------------------------------------------------------------------


template <int STAGES>
struct PairPCfg {
  static constexpr int A_BYTES = 16384;                    // 128 rows x 64 compressed bf16
  static constexpr int B_MAX = 32768;                      // up to 128 rows x 128 bf16 (two 64-wide boxes)
  static constexpr int E_BYTES = 2048;
  static constexpr int STAGE_BYTES = A_BYTES + B_MAX + E_BYTES;        // 50 KB (the B part is N / 2 rows)
  static constexpr int STAGING_BYTES = EPI_WARPS * 2048;   // per group of four epilogue warps: one [32 tokens][128 rows] bf16 tile
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 + 256;
};

template <int STAGES, bool CONV>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PAIR_THREADS, 1)
spmm_pair_persistent_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                            const __grid_constant__ CUtensorMap tmapE, const GemmParams p) {
  pdl_launch_dependents();
  using C = PairPCfg<STAGES>;
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
  const uint32_t nbuf = SP_N <= 240 ? 2u : 1u;            // accumulators in tensor memory
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
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    ptx::prefetch_tmap(&tmapE);
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
              a_row = tap * p.conv.rows_per_tap + m0;
              meta_row = a_row >> 7;
            }
            ptx::tma_load_2d_pair(a_s, &tmapA, a_col, a_row, bar);
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              int c0, dw, dh;
              bool valid;
              conv_k_coords(p.conv, kt, q, p.Kdim, c0, dw, dh, valid);
              ptx::tma_load_4d_pair(b_s + q * b_box, &tmapB, valid ? c0 : 0, cw0 + dw, ch0 + dh, valid ? cn0 : p.conv.NB, bar);
            }
            ptx::tma_load_2d_pair(b_s + C::B_MAX, &tmapE, 0, 2 * (meta_row * p.tiles_k_meta + meta_kt), bar);
            continue;
          }
          ptx::tma_load_2d_pair(a_s, &tmapA, kt * 64, m0, bar);
          ptx::tma_load_2d_pair(b_s, &tmapB, kt * 128, nrow, bar);
          ptx::tma_load_2d_pair(b_s + b_box, &tmapB, kt * 128 + 64, nrow, bar);
          ptx::tma_load_2d_pair(b_s + C::B_MAX, &tmapE, 0, 2 * (mt128 * p.tiles_k_meta + kt), bar);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && ptx::elect_one()) {
      const uint32_t idesc = ptx::idesc_bf16(256, SP_N, false, false, true);
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
          ptx::tmem_cp_128x128b_pair(tmem_meta, ptx::smem_desc(b_s + C::B_MAX, 0, 128, 0));
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t ad = ptx::smem_desc(a_s + kb * 32, 16, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + (kb >> 1) * b_box + (kb & 1) * 64, 16, 1024, 2);
            ptx::mma_sparse_pair(acc, ad, bd, tmem_meta + (kb & ~1), idesc | (uint32_t)(kb & 1), (kt | kb) != 0);
          }
          ptx::tc_commit_pair(empty_bar(s), 3);
        }
        if (ok) ptx::tc_commit_pair(tmem_full_bar(buf), 3);
      }
    }
  } else {
    // Each epilogue warp reads 32 accumulator rows (its TMEM lane quadrant); the four warps of a group share
    // one staging tile.
    const int q = warp & 3;
    const int eg = (warp - 2) >> 2;                        // EPI_WARPS / 4 groups of four warps take chunks in turn
    const uint32_t stg = staging + eg * 8192;
    uint16_t* outp = reinterpret_cast<uint16_t*>(p.out);
    uint32_t tcount = 0;
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
      const int nchunks = (CONV || (SP_N & 31) == 0) ? SP_N / 32 : SP_N / 16;
      if (CONV) {
        // accumulator columns [0, SP_N/2) are the pixels of box 2*tile_n, the rest those of box 2*tile_n + 1
        drain_chunks<32>(acc, eg, EPI_WARPS / 4, nchunks, false, release_bar, stg, 1 + eg, q, lane, p.Mdim - m0,
                         [&](int c, int t) -> uint16_t* {
          const int half = (32 * c) / (SP_N / 2);
          const int rr = 32 * c - half * (SP_N / 2) + t;
          int cw0, ch0, cn0;
          conv_box_origin(p.conv, 2 * tile_n + half, cw0, ch0, cn0);
          const int w = cw0 + (rr & (p.conv.wb - 1));
          const int h = ch0 + ((rr >> p.conv.lg_wb) & (p.conv.hb - 1));
          const int n = cn0 + (rr >> (p.conv.lg_wb + p.conv.lg_hb));
          if (w >= p.conv.W || h >= p.conv.H || n >= p.conv.NB) return nullptr;
          return outp + ((size_t)(n * p.conv.H + h) * p.conv.W + w) * p.Mdim + m0;
        });
      } else if ((SP_N & 31) == 0) {
        drain_chunks<32>(acc, eg, EPI_WARPS / 4, nchunks, false, release_bar, stg, 1 + eg, q, lane, p.Mdim - m0,
                         [&](int c, int t) -> uint16_t* {
          const int n = n0 + 32 * c + t;
          return n < p.Ndim ? outp + (size_t)n * p.Mdim + m0 : nullptr;
        });
      } else {
        drain_chunks<16>(acc, eg, EPI_WARPS / 4, nchunks, false, release_bar, stg, 1 + eg, q, lane, p.Mdim - m0,
                         [&](int c, int t) -> uint16_t* {
          const int n = n0 + 16 * c + t;
          return n < p.Ndim ? outp + (size_t)n * p.Mdim + m0 : nullptr;
        });
      }
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
// the same token tile, so the epilogue cannot overlap the next main loop; instead two groups of four
// epilogue warps per CTA drain the two accumulators side by side.  Metadata: columns 496..499 and 500..503.
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 accumulator 0, warps 6-9 accumulator 1.
// ------------------------------------------------------------------------------------------
constexpr int GEMM2M_THREADS = PAIR_THREADS;

template <int STAGES>
struct Pair2MCfg {
  static constexpr int A_BYTES = 16384;                    // per row tile: 128 rows x 64 compressed bf16
  static constexpr int B_MAX = 28672;                      // 112 rows x 128 bf16 (two 64-wide boxes), N <= 224
  static constexpr int E_BYTES = 2048;
  static constexpr int STAGE_BYTES = 2 * A_BYTES + B_MAX + 2 * E_BYTES;      // 64 KB
  static constexpr int STAGING_BYTES = EPI_WARPS * 2048;   // per group of four epilogue warps: one [32 tokens][128 rows] bf16 tile
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 + 256;
};

template <int STAGES>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM2M_THREADS, 1)
spmm_pair2m_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                   const __grid_constant__ CUtensorMap tmapE,
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
  const uint32_t tmem_empty_bar = bar_base + 8u * (2 * STAGES + 1);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(staging_ptr + C::STAGING_BYTES + 8 * (2 * STAGES + 2));
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
    ptx::mbar_init(tmem_empty_bar, 2 * EPI_WARPS);        // the epilogue warps of both CTAs of the pair
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
    ptx::prefetch_tmap(&tmapE);
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
      for (int tile = cluster_id; tile < num_tiles && ok; tile += num_clusters, ++tcount) {
        // both accumulators must have been drained by all sixteen epilogue warps of the pair
        if (!ptx::mbar_wait_bounded(tmem_empty_bar, (tcount & 1u) ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        ptx::tc_fence_after();
        for (int kt = 0; kt < num_kt; ++kt, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t a_s = base + s * C::STAGE_BYTES;
          const uint32_t b_s = a_s + 2 * C::A_BYTES;
          const uint32_t e_s = b_s + C::B_MAX;
          ptx::tmem_cp_128x128b_pair(tmem_meta, ptx::smem_desc(e_s, 0, 128, 0));
          ptx::tmem_cp_128x128b_pair(tmem_meta + 4u, ptx::smem_desc(e_s + C::E_BYTES, 0, 128, 0));
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
            for (int kb = 0; kb < 4; ++kb) {
              const uint64_t ad = ptx::smem_desc(a_s + mt * C::A_BYTES + kb * 32, 16, 1024, 2);
              const uint64_t bd = ptx::smem_desc(b_s + (kb >> 1) * b_box + (kb & 1) * 64, 16, 1024, 2);
              ptx::mma_sparse_pair(tmem_base + 256u * mt, ad, bd, tmem_meta + 4u * mt + (kb & ~1), idesc | (uint32_t)(kb & 1),
                                   (kt | kb) != 0);
            }
          }
          ptx::tc_commit_pair(empty_bar(s), 3);
        }
        if (ok) ptx::tc_commit_pair(tmem_full_bar, 3);
      }
    }
  } else {
    // warps 2-5 drain accumulator 0 (row tile 0), warps 6-9 accumulator 1; a warp reads its own
    // tensor-memory lane quadrant, a group shares one staging tile
    const int q = warp & 3;
    const int mt = (warp - 2) >> 2;                        // the group of four warps that drains accumulator mt
    const uint32_t stg = staging + mt * 8192;
    uint16_t* outp = reinterpret_cast<uint16_t*>(p.out);
    const uint32_t release_bar = ptx::mapa(tmem_empty_bar, 0);
    uint32_t tcount = 0;
    for (int tile = cluster_id; tile < num_tiles; tile += num_clusters, ++tcount) {
      int tile_m, tile_n;
      raster(tile, p.tiles_m, p.tiles_n, p.raster_group, tile_m, tile_n);
      const int m0 = mt128_of(tile_m, mt) * 128, n0 = tile_n * SP_N;
      bool ok = ptx::mbar_wait_bounded(tmem_full_bar, tcount & 1u, abort_flag, WAIT_BUDGET);
      ok = ptx::named_bar_and(1 + mt, 128, ok);            // the four warps of a group go on or give up together
      if (!ok) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
      const uint32_t acc = tmem_base + 256u * mt + ((uint32_t)(32 * q) << 16);
      drain_chunks<32>(acc, 0, 1, SP_N / 32, false, release_bar, stg, 1 + mt, q, lane, p.Mdim - m0,
                       [&](int c, int t) -> uint16_t* {
        const int n = n0 + 32 * c + t;
        return n < p.Ndim ? outp + (size_t)n * p.Mdim + m0 : nullptr;
      });
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
// Dense weight gradient on CTA pairs, persistent.  D[i, j] = sum_t dY[t, i] X[t, j]: both
// operands are read MN-major straight from the row-major activations (no transpose pass).  A
// pair owns a 256 x 256 tile; each CTA loads its 128 rows of dY^T and 128 of the 256 columns of
// X per stage (32 KB), the leader issues tcgen05.mma.cta_group::2, and the 512 tensor-memory
// columns hold TWO accumulators, so the epilogue of one tile (tensor memory -> registers ->
// 128-byte runs of fp32 in global memory) overlaps the main loop of the next.
// Work items are (tile, k-split) pairs; with more than one split the partial sums go to scratch.
// ------------------------------------------------------------------------------------------
template <int STAGES>
struct WgradCfg {
  static constexpr int A_BYTES = 16384, B_BYTES = 16384;     // 128 x 64 bf16 each, as two 64-wide boxes
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int TMEM_COLS = 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
};

// CONV: k tile kt is pixel box kt (64 pixels) of the NHWC tensors; the dy operand is that box, the
// x operand the same box shifted by the filter tap its 64 columns of dW belong to.
template <int STAGES, bool CONV>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
wgrad_pair_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                  const GemmParams p, int splits) {
  pdl_launch_dependents();
  using C = WgradCfg<STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar_base = base + STAGES * C::STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tmem_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tmem_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + 8 * (2 * STAGES + 4));
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
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
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
              ptx::tma_load_4d_pair(b_s + q * 8192, &tmapB, valid ? j - tap * p.conv.CB : 0, cw0 + tap % 3 - 1,
                                    ch0 + tap / 3 - 1, valid ? cn0 : p.conv.NB, bar);
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
  } else {
    const int q = warp & 3;
    uint32_t tcount = 0;
    for (int item = cluster_id; item < num_items; item += num_clusters, ++tcount) {
      int m0, n0, kt0, nkt, split;
      item_coords(item, m0, n0, kt0, nkt, split);
      const uint32_t buf = tcount & 1u;
      if (!ptx::mbar_wait_bounded(tmem_full_bar(buf), (tcount >> 1) & 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
      const int m = m0 + 32 * q + lane;
      float* out = reinterpret_cast<float*>(p.out) + (size_t)split * p.Mdim * p.Ndim;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + 256u * buf + ((uint32_t)(32 * q) << 16) + 32 * c, r);
        ptx::tmem_ld_wait();
        if (c == 7) {                                      // accumulator drained: release it
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_cluster(ptx::mapa(tmem_empty_bar(buf), 0));
        }
        const int nb = n0 + 32 * c;
        if (m < p.Mdim && nb < p.Ndim) {                  // Ndim % 32 == 0: a chunk is all in or all out
          float4* dst = reinterpret_cast<float4*>(out + (size_t)m * p.Ndim + nb);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                 __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
        }
      }
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
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 256;
};

template <int STAGES, bool CONV>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
wgrad_single_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
                    const GemmParams p, int splits) {
  pdl_launch_dependents();
  using C = WgradSingleCfg<STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar_base = base + STAGES * C::STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tmem_full_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tmem_empty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + 8 * (2 * STAGES + 4));
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
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
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
              ptx::tma_load_4d(b_s + q * 8192, &tmapB, valid ? j - tap * p.conv.CB : 0, cw0 + tap % 3 - 1, ch0 + tap / 3 - 1,
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
  } else {
    const int q = warp & 3;
    uint32_t tcount = 0;
    for (int item = blockIdx.x; item < num_items; item += gridDim.x, ++tcount) {
      int m0, n0, kt0, nkt, split;
      item_coords(item, m0, n0, kt0, nkt, split);
      const uint32_t buf = tcount & 1u;
      if (!ptx::mbar_wait_bounded(tmem_full_bar(buf), (tcount >> 1) & 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
      ptx::tc_fence_after();
      const int m = m0 + 32 * q + lane;
      float* out = reinterpret_cast<float*>(p.out) + (size_t)split * p.Mdim * p.Ndim;
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        uint32_t r[32];
        ptx::tmem_ld_32x32(tmem_base + 256u * buf + ((uint32_t)(32 * q) << 16) + 32 * c, r);
        ptx::tmem_ld_wait();
        if (c == 7) {                                      // accumulator drained: release it
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive_relaxed(tmem_empty_bar(buf));
        }
        const int nb = n0 + 32 * c;
        if (m < p.Mdim && nb < p.Ndim) {                  // Ndim % 32 == 0: a chunk is all in or all out
          float4* dst = reinterpret_cast<float4*>(out + (size_t)m * p.Ndim + nb);
#pragma unroll
          for (int j = 0; j < 8; ++j)
            dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                 __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
        }
      }
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
// dY[:, perm]: a streaming pass.  A CTA takes R token rows at a time (R = 4, or 2 for rows too
// long for a 4-row tile in shared memory): it reads
// them coalesced and stores them column-interleaved in shared memory (one 2R-byte word = the R
// rows' values of one column), so the gather costs one shared load per permuted column for all
// R rows; every thread then assembles eight consecutive permuted columns per row and writes
// them with one 16-byte store.
// ------------------------------------------------------------------------------------------
constexpr int PERMUTE_THREADS = 1024;

template <int R>
__global__ void __launch_bounds__(PERMUTE_THREADS)
permute_cols_kernel(const uint16_t* __restrict__ dY, const int32_t* __restrict__ perm, int T, int I,
                    uint16_t* __restrict__ dYp) {
  pdl_launch_dependents();
  pdl_wait();
  extern __shared__ uint32_t tile_w[];                   // R == 4: [I] x uint2, R == 2: [I] x uint32
  const int half = I >> 1;
  const int nthreads = (int)blockDim.x;                  // 256 .. 1024: short rows run more, smaller CTAs per SM
  for (int t0 = blockIdx.x * R; t0 < T; t0 += gridDim.x * R) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(dY) + (size_t)t0 * half;
    // four column chunks per trip: 4 R loads in flight per thread before any is consumed
    for (int c0 = threadIdx.x; c0 < half; c0 += 4 * nthreads) {
      uint32_t r[4][R];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * nthreads;
#pragma unroll
        for (int j = 0; j < R; ++j) r[u][j] = (c < half && t0 + j < T) ? __ldg(src + (size_t)j * half + c) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * nthreads;
        if (c < half) {
          if (R == 4) {
            reinterpret_cast<uint4*>(tile_w)[c] =
                make_uint4(__byte_perm(r[u][0], r[u][1], 0x5410), __byte_perm(r[u][2], r[u][R - 1], 0x5410),
                           __byte_perm(r[u][0], r[u][1], 0x7632), __byte_perm(r[u][2], r[u][R - 1], 0x7632));
          } else {
            reinterpret_cast<uint2*>(tile_w)[c] =
                make_uint2(__byte_perm(r[u][0], r[u][1], 0x5410), __byte_perm(r[u][0], r[u][1], 0x7632));
          }
        }
      }
    }
    __syncthreads();
    for (int k8 = threadIdx.x; k8 < (I >> 3); k8 += nthreads) {
      const int4 pa = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8);
      const int4 pb = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8 + 1);
      const int idx[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
      uint32_t lo[8], hi[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int i = min(max(idx[e], 0), I - 1);
        if (R == 4) {
          const uint2 v = reinterpret_cast<const uint2*>(tile_w)[i];
          lo[e] = v.x; hi[e] = v.y;
        } else {
          lo[e] = tile_w[i]; hi[e] = 0u;
        }
      }
      uint4 o[4];
      o[0] = make_uint4(__byte_perm(lo[0], lo[1], 0x5410), __byte_perm(lo[2], lo[3], 0x5410),
                        __byte_perm(lo[4], lo[5], 0x5410), __byte_perm(lo[6], lo[7], 0x5410));
      o[1] = make_uint4(__byte_perm(lo[0], lo[1], 0x7632), __byte_perm(lo[2], lo[3], 0x7632),
                        __byte_perm(lo[4], lo[5], 0x7632), __byte_perm(lo[6], lo[7], 0x7632));
      o[2] = make_uint4(__byte_perm(hi[0], hi[1], 0x5410), __byte_perm(hi[2], hi[3], 0x5410),
                        __byte_perm(hi[4], hi[5], 0x5410), __byte_perm(hi[6], hi[7], 0x5410));
      o[3] = make_uint4(__byte_perm(hi[0], hi[1], 0x7632), __byte_perm(hi[2], hi[3], 0x7632),
                        __byte_perm(hi[4], hi[5], 0x7632), __byte_perm(hi[6], hi[7], 0x7632));
#pragma unroll
      for (int j = 0; j < R; ++j)
        if (t0 + j < T) reinterpret_cast<uint4*>(dYp + (size_t)(t0 + j) * I)[k8] = o[j];
    }
    __syncthreads();
  }
}

// Short rows (I <= 1024): a row is at most 2 KB and stays in L1, so each thread simply gathers
// its eight permuted columns from global memory; rows are spread over all threads.
__global__ void __launch_bounds__(256)
permute_cols_small_kernel(const uint16_t* __restrict__ dY, const int32_t* __restrict__ perm, long long T, int I,
                          uint16_t* __restrict__ dYp) {
  pdl_launch_dependents();
  pdl_wait();
  const int per_row = I >> 3;
  const long long total = T * per_row;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const long long t = e / per_row;
    const int k8 = (int)(e - t * per_row);
    const uint16_t* row = dY + t * I;
    const int4 pa = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8);
    const int4 pb = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8 + 1);
    const int idx[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
    uint32_t v[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const uint32_t lo = __ldg(row + min(max(idx[2 * h], 0), I - 1));
      const uint32_t hi = __ldg(row + min(max(idx[2 * h + 1], 0), I - 1));
      v[h] = lo | (hi << 16);
    }
    reinterpret_cast<uint4*>(dYp + t * I)[k8] = make_uint4(v[0], v[1], v[2], v[3]);
  }
}

// Self-test of the bounded wait every GEMM role uses: one thread waits, with a budget of about
// a millisecond, on an mbarrier that nothing will ever complete.  The wait must give up, the kernel
// must report BIMASK_ETIMEOUT through the status word and return normally.
__global__ void wait_probe_kernel(long long budget_cycles, int32_t* __restrict__ status_word) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_barrier_init();
    const bool ok = ptx::mbar_wait_bounded(ptx::smem_u32(&bar), 0, &abort_flag, budget_cycles);
    if (!ok) atomicExch(status_word, (int32_t)BIMASK_ETIMEOUT);
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

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  });
  return fn;
}

// Encoding a tensor map costs a few microseconds on the host, which matters when a layer's
// kernels themselves run for ten.  A training loop passes the same buffers every step, so the
// encoded maps are kept in a small per-thread cache keyed by everything that went into them.
struct TmapKey {
  const void* ptr;
  uint64_t inner, outer, stride;
  uint32_t box_inner, box_outer;
  int dtype, swizzle;
  // rank 4 (NHWC activations: inner = channels, outer = W) when d2 != 0: extents H = d2, NB = d3,
  // densely packed (stride of H = W * stride, of NB = H * W * stride)
  uint64_t d2 = 0, d3 = 0;
  uint32_t box2 = 0, box3 = 0;
  bool operator==(const TmapKey& o) const {
    return ptr == o.ptr && inner == o.inner && outer == o.outer && stride == o.stride && box_inner == o.box_inner &&
           box_outer == o.box_outer && dtype == o.dtype && swizzle == o.swizzle && d2 == o.d2 && d3 == o.d3 &&
           box2 == o.box2 && box3 == o.box3;
  }
};

int encode_cached(CUtensorMap* m, const TmapKey& key) {
  constexpr int SLOTS = 32;
  static thread_local TmapKey keys[SLOTS];
  static thread_local CUtensorMap maps[SLOTS];
  static thread_local bool used[SLOTS] = {false};
  static thread_local int next = 0;
  for (int i = 0; i < SLOTS; ++i)
    if (used[i] && keys[i] == key) { *m = maps[i]; return BIMASK_OK; }
  EncodeTiledFn fn = get_encode_fn();
  BIMASK_REQUIRE(fn != nullptr, BIMASK_ECUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t dims[4] = {key.inner, key.outer, key.d2, key.d3};
  cuuint64_t strides[3] = {key.stride, key.stride * key.outer, key.stride * key.outer * key.d2};
  cuuint32_t box[4] = {key.box_inner, key.box_outer, key.box2, key.box3};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = fn(m, (CUtensorMapDataType)key.dtype, key.d2 ? 4 : 2, const_cast<void*>(key.ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, (CUtensorMapSwizzle)key.swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  BIMASK_REQUIRE(r == CUDA_SUCCESS, BIMASK_ECUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  keys[next] = key; maps[next] = *m; used[next] = true;
  next = (next + 1) % SLOTS;
  return BIMASK_OK;
}

int sm_count() {
  static thread_local int cached_dev = -1, cached = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev != cached_dev) {
    int n = 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) { cached = n; cached_dev = dev; }
  }
  return cached;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `outer` rows, box = 64 x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
int make_tmap(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_rows) {
  return encode_cached(m, TmapKey{ptr, inner, outer, inner * 2, 64, box_rows, (int)CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                  (int)CU_TENSOR_MAP_SWIZZLE_128B});
}

// The metadata image as a 2-D tensor of u32: 256 words per row, two rows per 2048-byte block.
int make_tmap_meta(CUtensorMap* m, const void* ptr, uint64_t blocks) {
  return encode_cached(m, TmapKey{ptr, 256, blocks * 2, 1024, 256, 2, (int)CU_TENSOR_MAP_DATA_TYPE_UINT32,
                                  (int)CU_TENSOR_MAP_SWIZZLE_NONE});
}

// 4-D bf16 map of an NHWC tensor (channels, W, H, NB) for loads of 64-channel pixel boxes, 128-byte swizzle.
int make_tmap_nhwc_load(CUtensorMap* m, const void* ptr, int CH, int W, int H, int NB, int wb, int hb, int nb) {
  TmapKey k{ptr, (uint64_t)CH, (uint64_t)W, (uint64_t)CH * 2, 64, (uint32_t)wb, (int)CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
            (int)CU_TENSOR_MAP_SWIZZLE_128B};
  k.d2 = (uint64_t)H; k.d3 = (uint64_t)NB; k.box2 = (uint32_t)hb; k.box3 = (uint32_t)nb;
  return encode_cached(m, k);
}

}  // namespace

// Generic 2-D tensor map without swizzle: `inner` contiguous elements of `elem_bytes` per row.
int make_tmap_plain(CUtensorMap* m, int dtype, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_inner,
                    uint32_t box_outer, uint32_t elem_bytes) {
  return encode_cached(m, TmapKey{ptr, inner, outer, inner * elem_bytes, box_inner, box_outer, dtype,
                                  (int)CU_TENSOR_MAP_SWIZZLE_NONE});
}

namespace {

// The dynamic shared-memory limit of a kernel is set once per (device, kernel): the call costs a microsecond or two
// on the host, which a layer step of ten short launches would notice.  A kernel is always launched with the same size.
template <typename K>
int set_smem_attr(K kernel, int bytes) {
  constexpr int SLOTS = 64;
  static std::atomic<const void*> done[16][SLOTS];       // [device][slot]; zero-initialised
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) dev = -1;
  const void* key = reinterpret_cast<const void*>(kernel);
  if (dev >= 0)
    for (int i = 0; i < SLOTS; ++i) {
      const void* seen = done[dev][i].load(std::memory_order_acquire);
      if (seen == key) return BIMASK_OK;
      if (seen == nullptr) break;
    }
  BIMASK_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  if (dev >= 0)
    for (int i = 0; i < SLOTS; ++i) {
      const void* expect = nullptr;
      if (done[dev][i].compare_exchange_strong(expect, key, std::memory_order_acq_rel) || expect == key) break;
    }
  return BIMASK_OK;
}

template <int N_TILE, int STAGES, bool SPARSE = true>
int run_single(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
               uint16_t* out, int32_t* status_word, cudaStream_t s) {
  using C = Cfg<N_TILE, STAGES, SPARSE>;
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap(&ta, vals, SPARSE ? (uint64_t)Kdim / 2 : (uint64_t)Kdim, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, N_TILE)) != BIMASK_OK) return rc;
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
  BIMASK_CUDA_OK(launch_pdl(kern, grid, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// Output-tile width of the CTA-pair 2:4 product.  Cost model in SM clocks, fitted to measurements: a tile's main
// loop takes 2 N clocks per 128-deep k tile; its epilogue (eight warps, two per lane quadrant) about 1100 clocks per
// 32-column chunk and warp, or 890 per 16-column chunk when N is not a multiple of 32; with N <= 240 the two
// overlap (two accumulators), with N = 256 they add up; narrower tiles re-read the compressed operand more often
// (L2 traffic), 0.3 % per column given up; the kernel's time is the number of passes over the clusters times the
// tile time.  (Short reductions are epilogue-bound: there a multiple of 32 wins.)
int choose_sparse_n(int pair_tiles_m, int Ndim, int k_tiles, int clusters) {
  int best_n = 256;
  double best = 1e30;
  for (int n = 256; n >= 160; n -= 16) {
    const long long tiles = (long long)pair_tiles_m * ((Ndim + n - 1) / n);
    const long long rounds = (tiles + clusters - 1) / clusters;
    const double mainloop = (double)k_tiles * 2.0 * n;
    const double epilogue = (n % 32 == 0) ? ((n / 32 + 1) / 2) * 1100.0 : ((n / 16 + 1) / 2) * 890.0;
    const double tile = n == 256 ? mainloop + epilogue : (mainloop > epilogue ? mainloop : epilogue);
    const double cost = (double)rounds * tile * (1.0 + 0.003 * (256 - n));
    if (cost < best) { best = cost; best_n = n; }
  }
  return best_n;
}

int run_sparse_pair_persistent(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim,
                               int Kdim, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  constexpr int STAGES = 3;
  using C = PairPCfg<STAGES>;
  CUtensorMap ta, tb, te;
  int rc;
  const int tiles_m = (Mdim + 127) / 128, tiles_k = (Kdim + 127) / 128;
  const int sms = sm_count();
  const int n_tile = choose_sparse_n((tiles_m + 1) / 2, Ndim, tiles_k, sms / 2);
  if ((rc = make_tmap(&ta, vals, (uint64_t)Kdim / 2, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, n_tile / 2)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_meta(&te, hw_meta, (uint64_t)tiles_m * tiles_k)) != BIMASK_OK) return rc;
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
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, te, p));
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
  CUtensorMap ta, tb, te;
  int rc;
  const int tiles_m = (Mdim + 127) / 128, tiles_k = (Kdim + 127) / 128;
  const int sms = sm_count();
  const int tiles_m512 = (tiles_m + 3) / 4;
  const int n_tile = choose_sparse_n_2m(tiles_m512, Ndim, tiles_k, sms / 2);
  if ((rc = make_tmap(&ta, vals, (uint64_t)Kdim / 2, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, n_tile / 2)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_meta(&te, hw_meta, (uint64_t)tiles_m * tiles_k)) != BIMASK_OK) return rc;
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
  p.raster_group = 4;
  const int total = p.tiles_m * p.tiles_n;
  const int clusters = total < sms / 2 ? total : sms / 2;
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, GEMM2M_THREADS, C::SMEM_BYTES, s, ta, tb, te, p));
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

int pow2_ceil(int v) { int p = 1; while (p < v) p <<= 1; return p; }
int log2_exact(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

// Pixel boxes of `tokens` tokens: as wide as the image allows (16 or 8), at least 32 tokens per image of the box.
void conv_boxes(ConvGeom& g, int tokens) {
  g.wb = g.W > 8 ? 16 : 8;
  int hb = tokens / g.wb;
  const int hp = pow2_ceil(g.H);
  if (hb > hp) hb = hp;
  if (hb < 32 / g.wb) hb = 32 / g.wb;
  g.hb = hb;
  g.nb = tokens / (g.wb * g.hb);
  g.lg_wb = log2_exact(g.wb);
  g.lg_hb = log2_exact(g.hb);
  g.tiles_w = (g.W + g.wb - 1) / g.wb;
  g.tiles_h = (g.H + g.hb - 1) / g.hb;
}

template <int N_TILE, int STAGES>
int run_conv_single(const uint16_t* vals, int a_rows, int a_kdim, const void* hw_meta, const uint16_t* tok, ConvGeom g,
                    int Mdim, int Kdim, int tiles_k_meta, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  using C = Cfg<N_TILE, STAGES, true>;
  conv_boxes(g, N_TILE);
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap(&ta, vals, (uint64_t)a_kdim / 2, (uint64_t)a_rows, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_nhwc_load(&tb, tok, g.CB, g.W, g.H, g.NB, g.wb, g.hb, g.nb)) != BIMASK_OK) return rc;
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
  BIMASK_CUDA_OK(launch_pdl(kern, grid, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int run_conv_pair(const uint16_t* vals, int a_rows, int a_kdim, const void* hw_meta, const uint16_t* tok, ConvGeom g,
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
  if ((rc = make_tmap_nhwc_load(&tb, tok, g.CB, g.W, g.H, g.NB, g.wb, g.hb, g.nb)) != BIMASK_OK) return rc;
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
  BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, PAIR_THREADS, C::SMEM_BYTES, s, ta, tb, te, p));
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
                     int I, uint16_t* out, int32_t* status_word, cudaStream_t s) {
  ConvGeom g{};
  g.mode = mode; g.H = H; g.W = W; g.NB = NB;
  const long long T = (long long)NB * H * W;
  int Mdim, Kdim, a_rows, a_kdim, tiles_k_meta;
  if (mode == 1) {
    g.CB = C; g.kt_per_tap = 0; g.rows_per_tap = 0;
    Mdim = I; Kdim = 9 * C; a_rows = I; a_kdim = 9 * C; tiles_k_meta = (9 * C + 127) / 128;
  } else {
    g.CB = I; g.kt_per_tap = (I + 127) / 128; g.rows_per_tap = C;
    Mdim = C; Kdim = 9 * g.kt_per_tap * 128; a_rows = 9 * C; a_kdim = I; tiles_k_meta = g.kt_per_tap;
  }
  if (Mdim > 128 && T > 128)
    return run_conv_pair(vals, a_rows, a_kdim, hw_meta, tok, g, Mdim, Kdim, tiles_k_meta, out, status_word, s);
  if (T > 128)
    return run_conv_single<256, 2>(vals, a_rows, a_kdim, hw_meta, tok, g, Mdim, Kdim, tiles_k_meta, out, status_word, s);
  return run_conv_single<128, 3>(vals, a_rows, a_kdim, hw_meta, tok, g, Mdim, Kdim, tiles_k_meta, out, status_word, s);
}

int launch_dense_nt(const uint16_t* A, const uint16_t* Bop, int Mdim, int Ndim, int Kdim, uint16_t* out,
                    int32_t* status_word, cudaStream_t s) {
  if (Ndim > 128) return run_single<256, 2, false>(A, nullptr, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  return run_single<128, 3, false>(A, nullptr, Bop, Mdim, Ndim, Kdim, out, status_word, s);
}

int launch_wait_probe(int32_t* status_word, cudaStream_t s) {
  BIMASK_CUDA_OK(launch_pdl(wait_probe_kernel, 1, 32, 0, s, 2000000ll, status_word));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_permute_cols(const uint16_t* dY, const int32_t* perm, int T, int I, uint16_t* dYp, cudaStream_t s) {
  if (I <= 1024) {
    const long long total = (long long)T * (I >> 3);
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    BIMASK_CUDA_OK(launch_pdl(permute_cols_small_kernel, (unsigned)blocks, 256, 0, s, dY, perm, (long long)T, I, dYp));
    count_launch();
    BIMASK_CUDA_OK(cudaGetLastError());
    return BIMASK_OK;
  }
  static bool attr_done = false;
  if (!attr_done) {
    BIMASK_CUDA_OK(cudaFuncSetAttribute(permute_cols_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    BIMASK_CUDA_OK(cudaFuncSetAttribute(permute_cols_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    attr_done = true;
  }
  const int R = (size_t)I * 8 <= 200 * 1024 ? 4 : 2;
  const size_t smem = (size_t)I * 2 * R;
  const int groups = (T + R - 1) / R;
  // a thread stages 16 row loads per trip and gathers 8 columns per trip: rows of I columns keep I / 8 threads busy
  const int threads = I >= 8192 ? PERMUTE_THREADS : I >= 4096 ? 512 : 256;
  int per_sm = (int)((200 * 1024) / smem);
  if (per_sm > 2048 / threads) per_sm = 2048 / threads;
  if (per_sm < 1) per_sm = 1;
  const int grid = groups < 148 * per_sm ? groups : 148 * per_sm;
  if (R == 4)
    BIMASK_CUDA_OK(launch_pdl(permute_cols_kernel<4>, grid, threads, smem, s, dY, perm, T, I, dYp));
  else
    BIMASK_CUDA_OK(launch_pdl(permute_cols_kernel<2>, grid, threads, smem, s, dY, perm, T, I, dYp));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

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

// The same for the implicit convolution: one k tile per 64-pixel box.
static ConvGeom conv_wgrad_geom(int NB, int H, int W, int C) {
  ConvGeom g{};
  g.mode = 1; g.H = H; g.W = W; g.NB = NB; g.CB = C;
  conv_boxes(g, 64);
  return g;
}

void wgrad_conv_plan(int NB, int H, int W, int C, int I, int* splits, int* k_tiles_per_split) {
  const ConvGeom g = conv_wgrad_geom(NB, H, W, C);
  wgrad_plan_k(g.tiles_w * g.tiles_h * ((NB + g.nb - 1) / g.nb), I, 9 * C, splits, k_tiles_per_split);
}

// dW[i, tap*C + c] = sum over pixels of dy[pixel, i] x[pixel + tap, c] without a column matrix (C % 64 == 0).
// partials: splits * I * 9C floats when wgrad_conv_plan gives more than one split.
int launch_wgrad_conv(const uint16_t* dy, const uint16_t* x, int NB, int H, int W, int C, int I, float* dW, float* partials,
                      int32_t* status_word, cudaStream_t s) {
  const ConvGeom g = conv_wgrad_geom(NB, H, W, C);
  const int boxes = g.tiles_w * g.tiles_h * ((NB + g.nb - 1) / g.nb);
  const int J = 9 * C;
  int splits, per;
  wgrad_plan_k(boxes, I, J, &splits, &per);
  constexpr int STAGES = 6;
  using Cf = WgradCfg<STAGES>;
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap_nhwc_load(&ta, dy, I, W, H, NB, g.wb, g.hb, g.nb)) != BIMASK_OK) return rc;
  if ((rc = make_tmap_nhwc_load(&tb, x, C, W, H, NB, g.wb, g.hb, g.nb)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv = g;
  p.hw_meta = nullptr; p.tiles_k_meta = 0;
  p.Mdim = I; p.Ndim = J; p.Kdim = boxes * 64;
  p.k_tiles_per_split = per;
  p.out = splits > 1 ? partials : dW;
  p.status_word = status_word;
  p.tiles_n = (J + 255) / 256;
  p.raster_group = 8;
  const int sms = sm_count();
  if (wgrad_uses_single(I)) {
    auto kern1 = wgrad_single_kernel<4, true>;
    if ((rc = set_smem_attr(kern1, WgradSingleCfg<4>::SMEM_BYTES)) != BIMASK_OK) return rc;
    p.tiles_m = 1;
    const int items = p.tiles_n * splits;
    BIMASK_CUDA_OK(launch_pdl(kern1, items < sms ? items : sms, GEMM_THREADS, WgradSingleCfg<4>::SMEM_BYTES, s, ta, tb, p, splits));
  } else {
    auto kern = wgrad_pair_kernel<STAGES, true>;
    if ((rc = set_smem_attr(kern, Cf::SMEM_BYTES)) != BIMASK_OK) return rc;
    p.tiles_m = ((I + 127) / 128 + 1) / 2;
    const int items = p.tiles_m * p.tiles_n * splits;
    const int clusters = items < sms / 2 ? items : sms / 2;
    BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, GEMM_THREADS, Cf::SMEM_BYTES, s, ta, tb, p, splits));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  if (splits > 1) {
    const long long n4 = (long long)I * J / 4;
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
                      int32_t* status_word, cudaStream_t s) {
  int nt, splits, per;
  wgrad_plan(T, I, J, &nt, &splits, &per);
  constexpr int STAGES = 6;
  using C = WgradCfg<STAGES>;
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap(&ta, dY, (uint64_t)I, (uint64_t)T, 64)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, X, (uint64_t)J, (uint64_t)T, 64)) != BIMASK_OK) return rc;
  GemmParams p;
  p.conv.mode = 0;
  p.hw_meta = nullptr; p.tiles_k_meta = 0;
  p.Mdim = I; p.Ndim = J; p.Kdim = T;
  p.k_tiles_per_split = per;
  p.out = splits > 1 ? partials : dW;
  p.status_word = status_word;
  p.tiles_n = (J + 255) / 256;
  p.raster_group = 8;
  const int sms = sm_count();
  if (wgrad_uses_single(I)) {
    auto kern1 = wgrad_single_kernel<4, false>;
    if ((rc = set_smem_attr(kern1, WgradSingleCfg<4>::SMEM_BYTES)) != BIMASK_OK) return rc;
    p.tiles_m = 1;
    const int items = p.tiles_n * splits;
    BIMASK_CUDA_OK(launch_pdl(kern1, items < sms ? items : sms, GEMM_THREADS, WgradSingleCfg<4>::SMEM_BYTES, s, ta, tb, p, splits));
  } else {
    auto kern = wgrad_pair_kernel<STAGES, false>;
    if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
    p.tiles_m = ((I + 127) / 128 + 1) / 2;
    const int items = p.tiles_m * p.tiles_n * splits;
    const int clusters = items < sms / 2 ? items : sms / 2;
    BIMASK_CUDA_OK(launch_pdl(kern, 2 * clusters, GEMM_THREADS, C::SMEM_BYTES, s, ta, tb, p, splits));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  if (splits > 1) {
    const long long n4 = (long long)I * J / 4;
    if ((rc = launch_splitk_reduce(partials, splits, n4, dW, s)) != BIMASK_OK) return rc;
  }
  return BIMASK_OK;
}

}  // namespace bimask
