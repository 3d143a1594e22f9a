// Forward mask + 2:4 packing (Eq. 4), backward mask + transposed packing (Eq. 11) and the
// re-ordering of the index metadata into the tensor core's TMEM image.
//
// All three are streaming kernels bound by HBM: every weight is read once per kernel with
// coalesced 128-bit (forward) or 128-byte-per-warp (backward, row gather) accesses, the
// selection is done on integer magnitude keys in registers, and the bit/nibble words are
// assembled with warp reductions / ballots so that every store is a full word.
#include "common.cuh"
#include "sm100_ptx.cuh"   // smem_u32
#include "mask_common.cuh"

namespace bimask {

namespace {

// ---------------------------------------------------------------------------------------
// Forward mask + pack.  W is treated as a flat stream of 4-element blocks (J % 32 == 0, so
// blocks, 32-column words and rows all nest).  A warp owns chunks of 256 blocks: eight
// coalesced float4 loads per lane go through an XOR-swizzled shared-memory stage so that each
// lane then owns EIGHT CONSECUTIVE blocks (one 32-column word): it builds the mask word and
// the code word locally, and stores its 32 bytes of values, with no cross-lane traffic.
// ---------------------------------------------------------------------------------------
constexpr int FWD_THREADS = 256;

// Optimizer update that ends the loop body of Algorithm 1, applied while the weights
// stream through the mask kernel so that the next iteration's forward mask costs no second pass
// over W.  float32, each product and sum rounded once, in this order (the updated weight decides
// a mask bit, so the operation order is part of the contract):
//   g = dW + weight_decay * W ;  mom = momentum * mom + g ;  W = W - lr * mom
template <bool N_IS_2, bool UPDATE>
__global__ void __launch_bounds__(FWD_THREADS)
fwd_mask_pack_kernel(const float4* __restrict__ W4, long long nblk, int N,
                     uint32_t* __restrict__ maskbits, uint4* __restrict__ vals4,
                     uint32_t* __restrict__ meta, uint16_t* __restrict__ hw16, int jwords, int pad_rows, SgdParams sgd) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ uint32_t lut[64];
  __shared__ float4 stage[FWD_THREADS / 32][256];
  if (threadIdx.x < 64) lut[threadIdx.x] = lut_entry(threadIdx.x, 0xFu, N);
  __syncthreads();
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const long long warp = (long long)blockIdx.x * (FWD_THREADS / 32) + wib;
  const long long nwarps = (long long)gridDim.x * (FWD_THREADS / 32);
  const long long nchunks = (nblk + 255) >> 8;
  float4* st = stage[wib];
  for (long long ch = warp; ch < nchunks; ch += nwarps) {
    const float4* src = W4 + (ch << 8);
    const int left = (int)min((long long)256, nblk - (ch << 8));      // multiple of 8
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int b = it * 32 + lane;
      float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
      if (UPDATE) {
        if (b < left) {
          const long long at = (ch << 8) + b;
          w = sgd.W4[at];
          const float4 dw = __ldg(sgd.dW4 + at);
          float4 m = sgd.mom4 ? sgd.mom4[at] : make_float4(0.f, 0.f, 0.f, 0.f);
          w.x = sgd_one(w.x, dw.x, m.x, sgd);
          w.y = sgd_one(w.y, dw.y, m.y, sgd);
          w.z = sgd_one(w.z, dw.z, m.z, sgd);
          w.w = sgd_one(w.w, dw.w, m.w, sgd);
          sgd.W4[at] = w;
          if (sgd.mom4) sgd.mom4[at] = m;
        }
      } else if (b < left) {
        w = __ldg(src + b);
      }
      st[b ^ ((b >> 3) & 7)] = w;
    }
    __syncwarp();
    uint32_t bits = 0, codes = 0, v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float4 w = st[lane * 8 + (j ^ (lane & 7))];
      const uint32_t k0 = mag_key(w.x), k1 = mag_key(w.y), k2 = mag_key(w.z), k3 = mag_key(w.w);
      const uint32_t e = lut[cmp6(k0, k1, k2, k3)];
      v[j] = slots<N_IS_2>(e, w.x, w.y, w.z, w.w, k0, k1, k2, k3);
      bits |= (e & 15u) << (4 * j);
      codes |= ((e >> 4) & 15u) << (4 * j);
    }
    __syncwarp();
    if (lane * 8 < left) {
      const long long word = (ch << 5) + lane;
      maskbits[word] = bits;
      meta[word] = codes;
      if (hw16) {
        const int r = (int)(word / jwords);
        scatter_hw(hw16, (jwords + 3) >> 2, r, (int)(word - (long long)r * jwords), codes);
      }
      vals4[2 * word] = make_uint4(v[0], v[1], v[2], v[3]);
      vals4[2 * word + 1] = make_uint4(v[4], v[5], v[6], v[7]);
    }
  }
  // padded operand (pad_rows = its row count): the image entries past the matrix
  if (hw16 && pad_rows)
    pad_hw_image(reinterpret_cast<uint32_t*>(hw16), pad_rows, jwords, (long long)blockIdx.x * FWD_THREADS + threadIdx.x,
                 (long long)gridDim.x * FWD_THREADS);
}

// ---------------------------------------------------------------------------------------
// Metadata re-order: canonical meta[rows][K/32] -> TMEM image.  One 2048-byte block per
// (128 rows, 128 k): 128 lanes x 4 columns of u32; lane L = m0 + 8*h + 16*m2 (m0 < 8, h < 2,
// m2 < 8), column c.  The word holds, for k in [128*kt + 32*c + 16*h, +16), the four codes
// of row m0 + 16*m2 in its low half and those of row m0 + 8 + 16*m2 in its high half.
// Rows / k beyond the matrix get the harmless code 0x4 (slots (0,1)), their values are 0.
// ---------------------------------------------------------------------------------------
__global__ void hw_meta_kernel(const uint32_t* __restrict__ meta, int rows, int kwords,
                               int tiles_k, long long total_lanes, uint4* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  // one thread per (tile, lane): the lane's four columns are one 16-byte store
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total_lanes) return;
  const int L = (int)(idx & 127);
  const long long tile = idx >> 7;
  const int kt = (int)(tile % tiles_k);
  const int mt = (int)(tile / tiles_k);
  const int m0 = L & 7, h = (L >> 3) & 1, m2 = L >> 4;
  const int r_lo = mt * 128 + m0 + 16 * m2;
  const int r_hi = r_lo + 8;
  const uint32_t sel = h ? 0x7632u : 0x5410u;            // low halves or high halves of (lo, hi)
  uint32_t o[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const int w = kt * 4 + c;
    uint32_t lo = 0x44444444u, hi = 0x44444444u;
    if (w < kwords) {
      if (r_lo < rows) lo = __ldg(meta + (long long)r_lo * kwords + w);
      if (r_hi < rows) hi = __ldg(meta + (long long)r_hi * kwords + w);
    }
    o[c] = __byte_perm(lo, hi, sel);
  }
  out[idx] = make_uint4(o[0], o[1], o[2], o[3]);
}

// ---------------------------------------------------------------------------------------
// Backward mask + transposed pack (Eq. 11).  Persistent CTAs walk tiles of 128 permuted rows x 64 CW columns
// (column tiles fastest, so the CTAs that run together read whole stretches of the same gathered rows).  Inside
// a tile warp w owns one item: the 32 rows (eight row-blocks) of row group w & 3 and the 32 CW columns of column
// item w >> 2.  Every warp runs its own three-deep ring of shared-memory stages filled by cp.async: the four row
// slices of row-block j+2 are in flight while row-block j is processed, also across the boundary between two
// tiles, and the ring costs no registers.
// Compute uses lane = column within each 32-column word (conflict-free shared loads).  The bit matrices at both
// ends are turned by a 32 x 32 shuffle transpose instead of per-block ballots: lane r loads the forward-mask word
// of its permuted row, after the transpose lane l holds the 32 candidate bits of its column, one nibble per
// row-block; the kept bits are collected the same way and transposed back into one backward-mask word per row.
// The operand being produced is transposed (row = column l of W, k contiguous), so a lane's results are 32 bytes
// of one operand row, a code word and a few mask bits: stored from the registers, every store instruction would
// touch 32 different 128-byte lines, and the load/store unit, not HBM, set the kernel's time.  The eight warps
// therefore put their results into a shared staging tile and the CTA writes it out in whole lines: 128 bytes per
// operand row, 16 bytes per code row and mask row, and the tile's 128 x 128 block of the tensor-memory image of
// the codes as one contiguous run.
// The selection table (1024 entries: six comparison bits x four candidate bits) is built once per CTA.
// CW = 2 (J a multiple of 64) for large matrices, CW = 1 for small ones (twice the tiles) and any J % 32 == 0.
// ---------------------------------------------------------------------------------------
constexpr int BM_WARPS = 8, BM_THREADS = 32 * BM_WARPS, BM_RING = 3, BM_CTAS_PER_SM = 4;
constexpr int BM_SV_PITCH = 36;                            // words per staged operand row: 32 + 4, conflict-free 16-byte accesses
template <int CW>
struct BMCfg {
  static constexpr int COLS = 64 * CW;                     // columns of a tile
  static constexpr int STAGE = 4 * 128 * CW;               // four row slices of 32 CW floats
  static constexpr int LUT_BYTES = 1024 * 4;
  static constexpr int RING_BYTES = BM_WARPS * BM_RING * STAGE;
  static constexpr int SV_BYTES = COLS * BM_SV_PITCH * 4;  // operand values [column][32 k pairs]
  static constexpr int SM_BYTES = 128 * 2 * CW * 4;        // backward-mask words [row][2 CW]
  static constexpr int SC_BYTES = COLS * 4 * 4;            // code words [column][4]
  static constexpr int SMEM = LUT_BYTES + RING_BYTES + SV_BYTES + SM_BYTES + SC_BYTES;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int CW>
__global__ void __launch_bounds__(BM_THREADS, BM_CTAS_PER_SM)
bwd_mask_kernel(const float* __restrict__ W, const uint32_t* __restrict__ maskbits_f,
                const int32_t* __restrict__ perm, int I, int J, int N,
                uint32_t* __restrict__ maskbits_b, uint32_t* __restrict__ vals_b,
                uint32_t* __restrict__ meta_b, uint32_t* __restrict__ hw32, int tiles_c, int n_tiles) {
  pdl_launch_dependents();
  using C = BMCfg<CW>;
  extern __shared__ __align__(128) uint8_t smem[];
  uint32_t* lut = reinterpret_cast<uint32_t*>(smem);
  uint8_t* ring_all = smem + C::LUT_BYTES;
  uint32_t* sv = reinterpret_cast<uint32_t*>(ring_all + C::RING_BYTES);
  uint32_t* sm = sv + C::SV_BYTES / 4;
  uint32_t* sc = sm + C::SM_BYTES / 4;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int e = threadIdx.x; e < 1024; e += BM_THREADS) lut[e] = lut_entry_signs(e & 63u, e >> 6, N);
  pdl_wait();                                              // the table needed no global memory
  __syncthreads();
  uint8_t* my_ring = ring_all + warp * BM_RING * C::STAGE;
  const uint32_t ring_u32 = ptx::smem_u32(my_ring);
  const int jwords = J >> 5;
  const int nrg = I >> 5;                                  // groups of 32 permuted rows
  const int items = jwords / CW;                           // column items of 32 CW columns
  const int rgi = warp & 3, cti = warp >> 2;               // this warp's row group and column item inside a tile
  const size_t vrow = (size_t)I >> 2;                      // u32 (bf16 pairs) per row of vals_b
  const size_t mrow = (size_t)I >> 5;

  // the gather of row-block j of an item whose 32 row indices the lanes hold in `rows`, into the stage at `soff`
  auto issue = [&](int rows, int item, int j, int soff) {
    // a row slice is 128 CW bytes = 8 CW lanes x 16 bytes: CW passes of 4 / CW rows each
#pragma unroll
    for (int ps = 0; ps < CW; ++ps) {
      const int m = ps * (4 / CW) + lane / (8 * CW), piece = lane % (8 * CW);
      const int r = __shfl_sync(0xFFFFFFFFu, rows, 4 * j + m);
      cp_async16(ring_u32 + soff + m * 128 * CW + 16 * piece, W + (size_t)r * J + item * 32 * CW + 4 * piece);
    }
    cp_async_commit();
  };
  auto load_rows = [&](int rgroup) { return checked_row(__ldg(perm + 32 * rgroup + lane), I, SITE_BWD_MASK_PERM); };
  auto load_fwd = [&](int rows, int item, uint32_t (&f)[CW]) {
    const uint32_t* src = maskbits_f + (size_t)rows * jwords + item * CW;
    if (CW == 2) { const uint2 t = __ldg(reinterpret_cast<const uint2*>(src)); f[0] = t.x; f[1] = t.y; }
    else f[0] = __ldg(src);
  };

  bool primed = false;                                     // the first two row-blocks of the coming item are in flight
  int off = 0;                                             // ring offset of the stage that holds the next row-block
  int rows_nxt = 0;
  uint32_t f_nxt[CW];
#pragma unroll
  for (int c = 0; c < CW; ++c) f_nxt[c] = 0u;
  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
    const int tr = tile / tiles_c, tc = tile - tr * tiles_c;
    const int rg = 4 * tr + rgi, item = 2 * tc + cti;
    const bool active = rg < nrg && item < items;          // warp uniform
    const int tile_n = tile + gridDim.x;
    const int tr_n = tile_n / tiles_c, tc_n = tile_n - tr_n * tiles_c;
    const int rg_n = 4 * tr_n + rgi, item_n = 2 * tc_n + cti;
    const bool active_n = tile_n < n_tiles && rg_n < nrg && item_n < items;
    if (active) {
      if (!primed) {
        rows_nxt = load_rows(rg);
        load_fwd(rows_nxt, item, f_nxt);
        off = 0;
        issue(rows_nxt, item, 0, 0);
        issue(rows_nxt, item, 1, C::STAGE);
      }
      const int rows_cur = rows_nxt;
      uint32_t cand[CW];                                   // candidate bits of this lane's columns, by row
#pragma unroll
      for (int c = 0; c < CW; ++c) cand[c] = transpose32(f_nxt[c], lane);
      if (active_n) rows_nxt = load_rows(rg_n);
      uint32_t vacc[CW][8];
      uint32_t cacc[CW], kacc[CW];
#pragma unroll
      for (int c = 0; c < CW; ++c) cacc[c] = kacc[c] = 0u;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        int ioff = off + 2 * C::STAGE;                     // the stage read in the previous step
        if (ioff >= BM_RING * C::STAGE) ioff -= BM_RING * C::STAGE;
        if (j + 2 < 8) issue(rows_cur, item, j + 2, ioff);
        else if (active_n) issue(rows_nxt, item_n, j + 2 - 8, ioff);   // the ring runs on into the next tile
        else cp_async_commit();                            // keep the group count uniform
        if (j == 4 && active_n) load_fwd(rows_nxt, item_n, f_nxt);
        cp_async_wait<2>();                                // row-block j has landed
        __syncwarp();
        const float* ws = reinterpret_cast<const float*>(my_ring + off);
        float w[4][CW];
#pragma unroll
        for (int m = 0; m < 4; ++m)
#pragma unroll
          for (int c = 0; c < CW; ++c) w[m][c] = ws[m * 32 * CW + 32 * c + lane];
        __syncwarp();                                      // all lanes have read the stage
        off += C::STAGE;
        if (off == BM_RING * C::STAGE) off = 0;
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          const uint32_t k0 = mag_key(w[0][c]), k1 = mag_key(w[1][c]), k2 = mag_key(w[2][c]), k3 = mag_key(w[3][c]);
          const uint32_t valid = (cand[c] >> (4 * j)) & 15u;
          const uint32_t e = lut[(valid << 6) | cmp6(k0, k1, k2, k3)];
          vacc[c][j] = slots_signs(e, w[0][c], w[1][c], w[2][c], w[3][c], k0, k1, k2, k3);
          kacc[c] |= ((e >> 16) & 15u) << (4 * j);
          cacc[c] |= ((e >> 24) & 15u) << (4 * j);
        }
      }
      primed = active_n;
      // results into the staging tile: 32 bytes of each operand row, its code word, and the mask words by row
#pragma unroll
      for (int c = 0; c < CW; ++c) {
        const int col = (cti * CW + c) * 32 + lane;
        uint4* dst = reinterpret_cast<uint4*>(sv + col * BM_SV_PITCH + 8 * rgi);
        dst[0] = make_uint4(vacc[c][0], vacc[c][1], vacc[c][2], vacc[c][3]);
        dst[1] = make_uint4(vacc[c][4], vacc[c][5], vacc[c][6], vacc[c][7]);
        sc[col * 4 + rgi] = cacc[c];
        sm[(32 * rgi + lane) * (2 * CW) + cti * CW + c] = transpose32(kacc[c], lane);
      }
    }
    __syncthreads();
    // ---- the CTA writes the tile out in whole lines ----
    const int rg0 = 4 * tr, item0 = 2 * tc;
    const int rgs_here = min(4, nrg - rg0), items_here = min(2, items - item0);
    const int col0 = item0 * 32 * CW, cols_here = items_here * 32 * CW;
#pragma unroll
    for (int it = 0; it < C::COLS * 8 / BM_THREADS; ++it) {
      const int idx = it * BM_THREADS + threadIdx.x;       // (column, 16-byte chunk of its 128 bytes)
      const int col = idx >> 3, chunk = idx & 7;
      if (col < cols_here && (chunk >> 1) < rgs_here)
        *reinterpret_cast<uint4*>(vals_b + (size_t)(col0 + col) * vrow + 8 * rg0 + 4 * chunk) =
            *reinterpret_cast<const uint4*>(sv + col * BM_SV_PITCH + 4 * chunk);
    }
    if (threadIdx.x < 128) {                               // backward-mask words of row rg0 * 32 + threadIdx.x
      const int row = threadIdx.x;
      if (row < 32 * rgs_here) {
        uint32_t* dst = maskbits_b + (size_t)(32 * rg0 + row) * jwords + item0 * CW;
        const uint32_t* src = sm + row * (2 * CW);
        if (CW == 2 && (jwords & 3) == 0) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
        else if ((jwords & 1) == 0 && items_here * CW >= 2) {
#pragma unroll
          for (int q = 0; q < CW; ++q)
            if (2 * q < items_here * CW) reinterpret_cast<uint2*>(dst)[q] = reinterpret_cast<const uint2*>(src)[q];
        } else {
          for (int q = 0; q < items_here * CW; ++q) dst[q] = src[q];
        }
      }
    } else {                                               // code words of operand row col0 + (threadIdx.x - 128)
      for (int col = threadIdx.x - 128; col < cols_here; col += 128) {
        uint32_t* dst = meta_b + (size_t)(col0 + col) * mrow + rg0;
        const uint32_t* src = sc + col * 4;
        if (rgs_here == 4 && (mrow & 3) == 0) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
        else for (int q = 0; q < rgs_here; ++q) dst[q] = src[q];
      }
    }
    if (hw32) {
      // tensor-memory image: the tile's codes fill a run of the 2048-byte block (operand rows col0 .., k words
      // rg0 ..): image lane L = m0 + 8 h + 16 m2 holds half h of the code words of rows m0 + 16 m2 (low 16 bits) and
      // m0 + 8 + 16 m2 (high 16 bits).  Entries past the matrix (padded shapes) are filled after the tile loop.
      uint32_t* blk = hw32 + ((size_t)(col0 >> 7) * ((I + 127) >> 7) + tr) * 512 + (col0 & 127) * 4;
#pragma unroll
      for (int it = 0; it < C::COLS * 4 / BM_THREADS; ++it) {
        const int idx = it * BM_THREADS + threadIdx.x;
        const int L = idx >> 2, kc = idx & 3;
        const int r_lo = (L & 7) + 16 * (L >> 4);
        if (r_lo < cols_here && kc < rgs_here) {
          const uint32_t lo = sc[r_lo * 4 + kc], hi = sc[(r_lo + 8) * 4 + kc];
          blk[idx] = __byte_perm(lo, hi, (L & 8) ? 0x7632u : 0x5410u);
        }
      }
    }
    __syncthreads();                                       // the staging tile is free again
  }
  cp_async_wait<0>();
  if (hw32 && ((I | J) & 127))                             // padded operand (J rows, I / 32 code words per row)
    pad_hw_image(hw32, J, I >> 5, (long long)blockIdx.x * BM_THREADS + threadIdx.x, (long long)gridDim.x * BM_THREADS);
}

}  // namespace

BIMASK_DEFINE_DEBUG_COLLECT(debug_collect_mask)

int launch_fwd_mask(const float* W, int I, int J, int N, uint32_t* maskbits, uint16_t* vals,
                    uint32_t* meta, void* hw_meta_or_null, cudaStream_t s) {
  uint16_t* hw16 = reinterpret_cast<uint16_t*>(hw_meta_or_null);
  const long long nblk = (long long)I * J / 4;
  const long long nchunks = (nblk + 255) >> 8;
  long long ctas = (nchunks + 7) / 8;
  if (ctas > 148 * 8) ctas = 148 * 8;
  if (ctas < 1) ctas = 1;
  const SgdParams none{nullptr, nullptr, nullptr, 0.f, 0.f, 0.f};
  const int pad_rows = (I % 128 || J % 128) ? I : 0;       // padded image: the kernel also fills the entries past the matrix
  if (N == 2)
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<true, false>, (unsigned)ctas, FWD_THREADS, 0, s,
        reinterpret_cast<const float4*>(W), nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, pad_rows, none));
  else
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<false, false>, (unsigned)ctas, FWD_THREADS, 0, s,
        reinterpret_cast<const float4*>(W), nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, pad_rows, none));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_sgd_fwd_mask(float* W, const float* dW, float* mom, int I, int J, int N, float lr, float momentum,
                        float weight_decay, uint32_t* maskbits, uint16_t* vals, uint32_t* meta,
                        void* hw_meta_or_null, cudaStream_t s) {
  const long long nblk = (long long)I * J / 4;
  uint16_t* hw16 = reinterpret_cast<uint16_t*>(hw_meta_or_null);
  long long ctas = ((nblk + 255) / 256 + (FWD_THREADS / 32) - 1) / (FWD_THREADS / 32);
  if (ctas > 148 * 8) ctas = 148 * 8;
  if (ctas < 1) ctas = 1;
  const SgdParams p{reinterpret_cast<float4*>(W), reinterpret_cast<const float4*>(dW), reinterpret_cast<float4*>(mom),
                    lr, momentum, weight_decay};
  const int pad_rows = (I % 128 || J % 128) ? I : 0;
  if (N == 2)
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<true, true>, (unsigned)ctas, FWD_THREADS, 0, s,
        nullptr, nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, pad_rows, p));
  else
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<false, true>, (unsigned)ctas, FWD_THREADS, 0, s,
        nullptr, nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, pad_rows, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_hw_meta(const uint32_t* meta, int rows, int K, void* hw_meta, cudaStream_t s) {
  const int tiles_m = (rows + 127) / 128, tiles_k = (K + 127) / 128;
  const long long total = (long long)tiles_m * tiles_k * 128;
  BIMASK_CUDA_OK(launch_pdl(hw_meta_kernel, (unsigned)((total + 255) / 256), 256, 0, s, meta, rows, K / 32, tiles_k, total,
                                                                 reinterpret_cast<uint4*>(hw_meta)));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_bwd_mask(const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                    int N, uint32_t* maskbits_b, uint16_t* vals_b, uint32_t* meta_b, void* hw_meta_or_null,
                    cudaStream_t s) {
  // tiles of 128 rows x 128 columns once they fill the resident CTAs, 128 x 64 (twice as many) otherwise
  const long long tiles_r = (I / 32 + 3) / 4;
  const bool wide = J % 64 == 0 && tiles_r * ((J / 64 + 1) / 2) >= (long long)BM_CTAS_PER_SM * 148;
  const int items = wide ? J / 64 : J / 32;
  const int tiles_c = (items + 1) / 2;
  const long long n_tiles = tiles_r * tiles_c;
  BIMASK_REQUIRE(n_tiles < (1ll << 30), BIMASK_EUNSUPPORTED, "bimask_bwd_mask: I * J = %lld is beyond the kernel's tile index",
                 (long long)I * J);
  const long long ctas = n_tiles < BM_CTAS_PER_SM * 148 ? n_tiles : BM_CTAS_PER_SM * 148;
  uint32_t* vals32 = reinterpret_cast<uint32_t*>(vals_b);
  uint32_t* hw32 = reinterpret_cast<uint32_t*>(hw_meta_or_null);
  if (wide) {
    if (int rc = set_smem_attr(bwd_mask_kernel<2>, BMCfg<2>::SMEM)) return rc;
    BIMASK_CUDA_OK(launch_pdl(bwd_mask_kernel<2>, (unsigned)ctas, BM_THREADS, BMCfg<2>::SMEM, s, W, maskbits_f, perm, I, J, N,
                              maskbits_b, vals32, meta_b, hw32, tiles_c, (int)n_tiles));
  } else {
    if (int rc = set_smem_attr(bwd_mask_kernel<1>, BMCfg<1>::SMEM)) return rc;
    BIMASK_CUDA_OK(launch_pdl(bwd_mask_kernel<1>, (unsigned)ctas, BM_THREADS, BMCfg<1>::SMEM, s, W, maskbits_f, perm, I, J, N,
                              maskbits_b, vals32, meta_b, hw32, tiles_c, (int)n_tiles));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace bimask
