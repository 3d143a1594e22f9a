// What the tensor-core kernels share: tile configurations, the convolution geometry, kernel parameters, the tile
// order, the accumulator drain of the 2:4 products, and the host helpers (tensor maps, SM count, shared-memory
// attribute) implemented in gemm_host.cu.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"
#include <cuda.h>
#include <cuda_bf16.h>
#include <atomic>

namespace bimask {


constexpr long long WAIT_BUDGET = 4000000000ll;      // ~2 s of SM clocks
constexpr int GEMM_THREADS = 192;                    // warp 0 TMA, warp 1 MMA, warps 2-5 epilogue
// The sparse kernels that drain bf16 results use eight epilogue warps (two groups of four, one warp per
// tensor-memory lane quadrant, taking alternate column chunks): products with a short reduction are bound by
// that drain, not by the tensor pipe.
constexpr int EPI_WARPS = 8;
// One more warp per group of four epilogue warps issues the tensor stores of the group's staged chunks (see
// drain_chunks_tma / store_chunks): a tensor store costs its issuing thread a few hundred clocks, which the warps
// that drain tensor memory should not wait for.
constexpr int EPI_GROUPS = EPI_WARPS / 4;
constexpr int PAIR_THREADS = 64 + 32 * EPI_WARPS + 32 * EPI_GROUPS;
// Epilogue staging: per group NT tiles of [32 tokens][128 rows] bf16 (8 KB each), and per group NT "staged" plus NT
// "freed" mbarriers, kept EPI_BAR_OFFSET bytes into the kernels' barrier area.
__host__ __device__ constexpr int epi_staging_bytes(int nt) { return EPI_GROUPS * nt * 8192; }
constexpr uint32_t EPI_BAR_OFFSET = 128;


template <int N_TILE, int STAGES, bool SPARSE = true>
struct Cfg {
  static constexpr int M_TILE = 128;
  static constexpr int K_TILE = 128;                             // logical reduction elements per stage
  static constexpr int A_BYTES = SPARSE ? 16384 : 32768;         // 128 rows x 64 compressed, or x 128 dense, bf16
  static constexpr int B_BYTES = N_TILE * K_TILE * 2;
  static constexpr int E_BYTES = SPARSE ? 2048 : 0;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
  static constexpr int META_COLS = SPARSE ? 4 : 0;
  static constexpr int EPI_NT = SPARSE ? 3 : 2;                  // staging tiles per epilogue group (the dense stages leave room for two)
  static constexpr int TMEM_COLS = (N_TILE + META_COLS) <= 128 ? 128 : (N_TILE + META_COLS) <= 256 ? 256 : 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */ +
                                    epi_staging_bytes(EPI_NT) /* epilogue staging */;
};

// A 3x3 convolution as an implicit GEMM: the token operand is an NHWC tensor and a "tile of
// tokens" is a box of wb x hb pixels of nb images, fetched with one 4-D tensor load per 64
// channels, shifted by the filter tap the k index belongs to (pixels outside the image read 0).
//   mode 1 (forward, Eq. 3):        k = (tap, c);  B = x,   shift (+kw-1, +kh-1)
//   mode 2 (input gradient, Eq. 10): k = (tap, i');  B = dy[:, perm], shift (1-kw, 1-kh); the rows of
//           the 2:4 operand for tap (kh, kw) are (kh*3+kw)*C + c.
struct ConvGeom {
  int mode;                 // 0: plain matrix operand
  int H, W, NB;             // grid of the tokens (the convolution's OUTPUT pixels)
  int stride;               // mode 1 / weight gradient: input pixel of output pixel (h, w), tap (kh, kw) is
                            // (stride * h + kh - 1, stride * w + kw - 1); the input tensor map strides by it
  int CB;                   // channels of the token operand (x: C; dy: I)
  int wb, hb, nb;           // pixel box of one load: wb * hb * nb tokens (powers of two)
  int lg_wb, lg_hb;         // their logarithms
  int tiles_w, tiles_h;     // boxes per image
  int kt_per_tap;           // mode 2: 128-wide k tiles per filter tap (I / 128)
  int rows_per_tap;         // mode 2: rows of the 2:4 operand per tap (C)
  // mode 2: the filter taps this launch sums over, in k order: tap id (kh * 3 + kw, selects the operand rows) and the
  // shift of the dy box.  Stride 1: all nine, shift (1 - kw, 1 - kh).  Stride 2: the input pixels of one parity class
  // (h % 2, w % 2) receive gradient through the taps with kh = h + 1 and kw = w + 1 (mod 2) only -- one, two, two and
  // four taps for the four classes -- from dy pixel ((h + 1 - kh) / 2, (w + 1 - kw) / 2); the token grid is then the
  // class's sub-grid and the results go to every second pixel of dx.
  signed char tap_id[9], tap_dw[9], tap_dh[9];
  int out_step, out_h0, out_w0, out_H, out_W;   // token (h, w) is stored at pixel (out_step * h + out_h0, out_step * w + out_w0) of out_H x out_W
};

// Where the results of token pixel (n, h, w) go: element offset of its first channel in the NHWC output.
__device__ __forceinline__ size_t conv_out_pixel(const ConvGeom& g, int n, int h, int w) {
  return ((size_t)n * g.out_H + (g.out_step * h + g.out_h0)) * g.out_W + (g.out_step * w + g.out_w0);
}

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
    dh = g.tap_dh[tap];
    dw = g.tap_dw[tap];
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
  int n_tile;               // pair kernel: output columns per tile (multiple of 32, <= 256)
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

// Epilogue of the 2:4 products, form with per-lane global stores (used where a token's address is not affine in
// its index: the pixel boxes of the implicit convolution; drain_chunks_tma below is the form for plain matrices).
// The accumulator holds D[row][token] (row = tensor-memory lane), the result is
// stored token-major, so a chunk of W tokens x the CTA's 128 rows is transposed on its way out by a GROUP of four
// warps, one per tensor-memory lane quadrant:
//   tensor memory -> registers in the accumulator-fragment layout (two 16-lane loads per warp) -> bf16 pairs ->
//   stmatrix.trans into one of the group's two staging tiles [token][128 rows] (256-byte rows; the 16-byte unit
//   index is XOR-ed with the token index mod 8, so the eight rows of a matrix fall into eight different bank
//   groups) -> named barrier -> each warp reads W/4 whole token rows back and writes them with 16-byte stores,
//   256 contiguous bytes per token (whole 128-byte lines).
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

// `dst`: this lane's row address for token group 0 (see drain_chunks); token group g is GROUP_BYTES further (eight
// token rows of the staging tile).
template <int W, uint32_t GROUP_BYTES = 2048u>
__device__ __forceinline__ void epi_stage(const uint32_t (&r)[W], uint32_t dst) {
#pragma unroll
  for (int g = 0; g < W / 8; ++g)
    ptx::stmatrix_x4_trans(dst + GROUP_BYTES * g, pack_bf16(r[4 * g], r[4 * g + 1]), pack_bf16(r[4 * g + 2], r[4 * g + 3]),
                           pack_bf16(r[W / 2 + 4 * g], r[W / 2 + 4 * g + 1]),
                           pack_bf16(r[W / 2 + 4 * g + 2], r[W / 2 + 4 * g + 3]));
}

// The staging and store half of the drain, shared by the two schedules below: state of one warp of a group.
// `stg`: the group's two staging tiles (2 x W * 256 bytes, 1 KB aligned); `bar_id`: its named barrier.  Every tile
// of the accumulator loop starts with the first staging tile: the callers synchronise the group between two tiles
// (the barrier on which the group agrees that the next accumulator is ready), so the last read-back of one tile is
// over before the next one stages.
// row_of(c, t) returns where token t of chunk c starts in the result (the CTA's first row), or nullptr when that
// token lies outside; rows_valid = how many of the CTA's 128 rows exist (a multiple of 32).
template <int W>
struct DrainWarp {
  uint32_t stg, bar_id, dst, parity;
  int q, lane, unit;
  bool unit_ok;
  __device__ __forceinline__ DrainWarp(uint32_t stg_, uint32_t bar_id_, int q_, int lane_, int rows_valid)
      : stg(stg_), bar_id(bar_id_), parity(0), q(q_), lane(lane_), unit(lane_ & 15), unit_ok(8 * (lane_ & 15) < rows_valid) {
    // stmatrix: lane 8 i + k addresses token k (of a group of eight) of matrix i = rows 32 q + 8 i .. + 7, i.e. unit
    // 4 q + i of the token's 256-byte row
    dst = stg + (uint32_t)(lane & 7) * 256u + ((((uint32_t)(4 * q) + ((uint32_t)lane >> 3)) ^ ((uint32_t)lane & 7u)) << 4);
  }
  // reading back: this warp owns tokens (W/4) q .. (W/4) q + W/4 - 1; per step lanes 0-15 take one token, lanes 16-31
  // the next, 16 bytes (eight rows) per lane
  template <typename RowOf>
  __device__ __forceinline__ void emit(const uint32_t (&r)[W], int c, RowOf& row_of) {
    // Two tiles, one barrier per chunk: a tile is staged again two chunks later, and between the read-back of this
    // chunk and that staging every warp of the group passes the barrier of the chunk in between.
    const uint32_t tile = parity * (uint32_t)(W * 256);
    parity ^= 1u;
    uint16_t* row[W / 8];                                 // where this lane's tokens go: worked out ahead of the barrier
#pragma unroll
    for (int i = 0; i < W / 8; ++i) {
      uint16_t* r0 = row_of(c, (W / 4) * q + 2 * i + (lane >> 4));
      row[i] = (r0 != nullptr && unit_ok) ? r0 + 8 * unit : nullptr;
    }
    epi_stage<W>(r, dst + tile);
    ptx::named_bar_sync(bar_id, 128);
    uint4 v[W / 8];
#pragma unroll
    for (int i = 0; i < W / 8; ++i) {
      const int t = (W / 4) * q + 2 * i + (lane >> 4);
      v[i] = ptx::ld_shared_v4(stg + tile + (uint32_t)t * 256u + (((uint32_t)unit ^ ((uint32_t)t & 7u)) << 4));
    }
#pragma unroll
    for (int i = 0; i < W / 8; ++i)
      if (row[i] != nullptr) *reinterpret_cast<uint4*>(row[i]) = v[i];
  }
};

// After its last tensor-memory read a warp arrives once on `release_bar` (0: nobody waits for the accumulator).
__device__ __forceinline__ void release_accumulator(uint32_t release_bar, int lane) {
  if (release_bar != 0u) {
    ptx::tc_fence_before();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive_cluster(release_bar);
  }
}

// The accumulator loop shared by the two write-out forms below: chunks c0, c0 + cstep, ... (< nchunks) of one
// accumulator (column of chunk c: W * c) go through emit(registers, c); one chunk is converted and written while the
// tensor-memory load of the next is in flight.
template <int W, typename Emit>
__device__ __forceinline__ void drain_loop(uint32_t acc, int c0, int cstep, int nchunks, bool zero, uint32_t release_bar,
                                           int lane, Emit&& emit) {
  uint32_t ra[W], rb[W];
  epi_load<W>(acc + W * c0, ra, zero);
#pragma unroll 1
  for (int c = c0; c < nchunks; c += 2 * cstep) {
    if (!zero) ptx::tmem_ld_wait();
    const bool more1 = c + cstep < nchunks;
    if (more1) epi_load<W>(acc + W * (c + cstep), rb, zero); else release_accumulator(release_bar, lane);
    emit(ra, c);
    if (!more1) break;
    if (!zero) ptx::tmem_ld_wait();
    if (c + 2 * cstep < nchunks) epi_load<W>(acc + W * (c + 2 * cstep), ra, zero); else release_accumulator(release_bar, lane);
    emit(rb, c + cstep);
  }
}

// Drains chunks c0, c0 + cstep, ... (< nchunks) of one accumulator; called by the four warps of a group with the
// same arguments except `acc` (the warp's lane quadrant q = warp % 4).  Results leave through per-lane 16-byte
// stores to addresses that row_of supplies (any token-to-address mapping: the implicit convolution's pixel boxes).
template <int W, typename RowOf>
__device__ __forceinline__ void drain_chunks(uint32_t acc, int c0, int cstep, int nchunks, bool zero, uint32_t release_bar,
                                             uint32_t stg, uint32_t bar_id, int q, int lane, int rows_valid, RowOf&& row_of) {
  if (c0 >= nchunks) { release_accumulator(release_bar, lane); return; }
  DrainWarp<W> d(stg, bar_id, q, lane, rows_valid);
  drain_loop<W>(acc, c0, cstep, nchunks, zero, release_bar, lane, [&](const uint32_t (&r)[W], int c) { d.emit(r, c, row_of); });
}

// The same drain for results that are a plain [token][row] matrix: a chunk leaves as two tensor stores (TMA) of
// W tokens x 64 rows, straight from a staging tile, issued by the group's STORE thread (store_chunks below) so
// that the draining warps never wait for a store to be issued.  A staging tile is two halves [W tokens][64 rows] of
// 128-byte token rows in the 128-byte-swizzled layout of the tensor map (16-byte unit index XOR token index mod 8
// -- the same XOR that keeps stmatrix free of bank conflicts).  The group's NT tiles are used in turn over the
// whole kernel (chunk number u of the group -> tile u % NT); two mbarriers per tile hand it back and forth:
//   staged[t]  (4 arrivals: one per draining warp, after stmatrix and a proxy fence)   drain -> store thread
//   freed[t]   (1 arrival: the store thread, once the tile's stores have read it)       store thread -> drain
// `bars`: the group's barriers (NT staged, then NT freed); `u`: the group's chunk counter, carried from call to
// call.  Returns false when a wait ran out of budget (the caller raises the abort flag).
template <int NT>
__device__ __forceinline__ void epi_bars_init(uint32_t bar_area) {
#pragma unroll
  for (int g = 0; g < EPI_GROUPS; ++g)
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      ptx::mbar_init(bar_area + EPI_BAR_OFFSET + 8u * (g * 2 * NT + t), 4);
      ptx::mbar_init(bar_area + EPI_BAR_OFFSET + 8u * (g * 2 * NT + NT + t), 1);
    }
}
template <int NT>
__device__ __forceinline__ uint32_t epi_bars_of(uint32_t bar_area, int g) { return bar_area + EPI_BAR_OFFSET + 8u * (g * 2 * NT); }

template <int W, int NT>
__device__ __forceinline__ bool drain_chunks_tma(uint32_t acc, int c0, int cstep, int nchunks, bool zero, uint32_t release_bar,
                                                 uint32_t stg, uint32_t bars, uint32_t& u, int q, int lane,
                                                 volatile int* abort_flag) {
  if (c0 >= nchunks) { release_accumulator(release_bar, lane); return true; }
  // stmatrix: lane 8 i + k addresses token k (of a group of eight) of matrix i = rows 32 q + 8 i .. + 7, i.e. 16-byte
  // unit 4 (q & 1) + i of the token's row in half q >> 1
  const uint32_t dst = stg + (uint32_t)(q >> 1) * (uint32_t)(W * 128) + (uint32_t)(lane & 7) * 128u +
                       ((((uint32_t)(4 * (q & 1)) + ((uint32_t)lane >> 3)) ^ ((uint32_t)lane & 7u)) << 4);
  bool ok = true;
  drain_loop<W>(acc, c0, cstep, nchunks, zero, release_bar, lane, [&](const uint32_t (&r)[W], int) {
    const uint32_t slot = u % NT, use = u / NT;
    ++u;
    if (use > 0 && ok) ok = ptx::mbar_wait_bounded(bars + 8u * (NT + slot), (use - 1u) & 1u, abort_flag, WAIT_BUDGET);
    epi_stage<W, 1024u>(r, dst + slot * 8192u);
    ptx::fence_proxy_async();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(bars + 8u * slot);
  });
  return ok;
}

// The store thread's side of drain_chunks_tma, called with the same chunk sequence: waits for a staged tile, issues
// its stores (rows and tokens outside the result are clipped by the tensor map, extent Mdim x Ndim; a store that
// would start outside is not issued), and hands back the tile of the previous chunk once its stores have read it.
// x0: first row of the CTA's 128; y0: first token of chunk 0.  After its last call the thread runs store_finish().
template <int W, int NT>
__device__ __forceinline__ bool store_chunks(const CUtensorMap* tmapD, int c0, int cstep, int nchunks, uint32_t stg,
                                             uint32_t bars, uint32_t& u, int x0, int y0, int Mdim, int Ndim,
                                             volatile int* abort_flag) {
  for (int c = c0; c < nchunks; c += cstep) {
    const uint32_t slot = u % NT, use = u / NT;
    if (!ptx::mbar_wait_bounded(bars + 8u * slot, use & 1u, abort_flag, WAIT_BUDGET)) return false;
    const int y = y0 + W * c;
    if (y < Ndim && x0 < Mdim) {
      ptx::tma_store_2d(tmapD, x0, y, stg + slot * 8192u);
      if (x0 + 64 < Mdim) ptx::tma_store_2d(tmapD, x0 + 64, y, stg + slot * 8192u + (uint32_t)(W * 128));
    }
    ptx::bulk_commit();
    if (u > 0) {
      ptx::bulk_wait_read<1>();
      ptx::mbar_arrive(bars + 8u * (NT + (u - 1u) % NT));
    }
    ++u;
  }
  return true;
}
// Shared memory must outlive the stores that read it.
__device__ __forceinline__ void store_finish() { ptx::bulk_wait_read<0>(); }

// ---- host helpers (gemm_host.cu) -----------------------------------------------------------
int sm_count();
// 2-D bf16 tensor map: `inner` contiguous elements per row, `outer` rows, box = 64 x box_rows, 128-byte swizzle,
// out-of-range elements read as zero.
int make_tmap(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_rows);
// The metadata image as a 2-D tensor of u32: 256 words per row, two rows per 2048-byte block.
int make_tmap_meta(CUtensorMap* m, const void* ptr, uint64_t blocks);
// fp32 [planes][rows][inner] for stores of 32 x 128 boxes (the dense product's result or its split-K partial sums).
int make_tmap_f32_store(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t rows, uint64_t planes);
// 4-D bf16 map of an NHWC tensor (channels, W, H, NB) for loads of 64-channel pixel boxes, 128-byte swizzle.
// estride 2: a box takes every second pixel along W and H (wb x hb pixels all the same).
int make_tmap_nhwc_load(CUtensorMap* m, const void* ptr, int CH, int W, int H, int NB, int wb, int hb, int nb, int estride = 1);

// ---- pixel boxes of the implicit convolution ------------------------------------------------
inline int pow2_ceil(int v) { int p = 1; while (p < v) p <<= 1; return p; }
inline int log2_exact(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

// Pixel boxes of `tokens` tokens: as wide as the image allows (16 or 8), at least 32 tokens per image of the box.
inline void conv_boxes(ConvGeom& g, int tokens) {
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

}  // namespace bimask
