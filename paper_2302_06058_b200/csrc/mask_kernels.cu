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

// Optimizer update of Algorithm 1 ("update via the SGD optimizer"), applied while the weights
// stream through the mask kernel so that the next iteration's forward mask costs no second pass
// over W.  float32, each product and sum rounded once, in this order (the updated weight decides
// a mask bit, so the operation order is part of the contract):
//   g = dW + weight_decay * W ;  mom = momentum * mom + g ;  W = W - lr * mom
struct SgdParams {
  float4* W4;            // read and written
  const float4* dW4;
  float4* mom4;          // nullptr: momentum buffer treated as zero and not stored
  float lr, momentum, weight_decay;
};

__device__ __forceinline__ float sgd_one(float w, float dw, float& m, const SgdParams& p) {
  const float g = __fadd_rn(dw, __fmul_rn(p.weight_decay, w));
  m = __fadd_rn(__fmul_rn(p.momentum, m), g);
  return __fsub_rn(w, __fmul_rn(p.lr, m));
}

template <bool N_IS_2, bool UPDATE>
__global__ void __launch_bounds__(FWD_THREADS)
fwd_mask_pack_kernel(const float4* __restrict__ W4, long long nblk, int N,
                     uint32_t* __restrict__ maskbits, uint4* __restrict__ vals4,
                     uint32_t* __restrict__ meta, uint16_t* __restrict__ hw16, int jwords, SgdParams sgd) {
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
        scatter_hw(hw16, jwords >> 2, r, (int)(word - (long long)r * jwords), codes);
      }
      vals4[2 * word] = make_uint4(v[0], v[1], v[2], v[3]);
      vals4[2 * word + 1] = make_uint4(v[4], v[5], v[6], v[7]);
    }
  }
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
// Backward mask + transposed pack (Eq. 11).  The unit of work is one warp item: 32 permuted rows (eight
// row-blocks) x 32 CW columns.  Persistent CTAs; every warp walks its own items (column tiles fastest, so the warps
// that run together read whole stretches of the same gathered rows) with its own four-deep ring of shared-memory
// stages filled by cp.async: the four row slices of row-block j+3 are in flight while row-block j is processed,
// also across the boundary between two items, and the ring costs no registers.
// Compute uses lane = column within each 32-column word (conflict-free shared loads).  The bit matrices at both
// ends are turned by a 32 x 32 shuffle transpose instead of per-block ballots: lane r loads the forward-mask word
// of its permuted row, after the transpose lane l holds the 32 candidate bits of its column, one nibble per
// row-block; the kept bits are collected the same way and transposed back into one backward-mask word per row.
// The operand being produced is transposed (row = column l of W, k contiguous): a lane keeps the eight
// consecutive k results of its columns in registers and writes them as full 32-byte sectors; the two halves of
// a code word go to the tensor-memory image as 32-bit words shared with the lane eight columns away.
// The selection table (1024 entries: six comparison bits x four candidate bits) is built once per CTA.
// CW = 2 (J a multiple of 64) for large matrices, CW = 1 for small ones (twice the items) and any J % 32 == 0.
// ---------------------------------------------------------------------------------------
constexpr int BM_WARPS = 8, BM_THREADS = 32 * BM_WARPS, BM_RING = 4, BM_CTAS_PER_SM = 4;
template <int CW>
struct BMCfg {
  static constexpr int STAGE = 4 * 128 * CW;               // four row slices of 32 CW floats
  static constexpr int LUT_BYTES = 1024 * 8;
  static constexpr int SMEM = LUT_BYTES + BM_WARPS * BM_RING * STAGE;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Transpose of a 32 x 32 bit matrix held one row per lane (bit b of lane r = element (r, b)): five exchange
// stages, each swapping the off-diagonal quadrants of every 2s x 2s block; afterwards lane c holds column c.
__device__ __forceinline__ uint32_t transpose32(uint32_t x, int lane) {
  {
    const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, 16);
    x = __byte_perm(x, y, (lane & 16) ? 0x3276u : 0x5410u);
  }
  {
    const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, 8);
    x = __byte_perm(x, y, (lane & 8) ? 0x3715u : 0x6240u);
  }
#pragma unroll
  for (int s = 4; s >= 1; s >>= 1) {
    const uint32_t m = s == 4 ? 0x0F0F0F0Fu : s == 2 ? 0x33333333u : 0x55555555u;
    const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, s);
    const bool low = (lane & s) == 0;                      // this lane keeps its low half of every 2s group
    const uint32_t keep = low ? m : ~m;
    const uint32_t moved = low ? (y << s) : (y >> s);
    x = (x & keep) | (moved & ~keep);
  }
  return x;
}

template <int CW>
__global__ void __launch_bounds__(BM_THREADS, BM_CTAS_PER_SM)
bwd_mask_kernel(const float* __restrict__ W, const uint32_t* __restrict__ maskbits_f,
                const int32_t* __restrict__ perm, int I, int J, int N,
                uint32_t* __restrict__ maskbits_b, uint32_t* __restrict__ vals_b,
                uint32_t* __restrict__ meta_b, uint32_t* __restrict__ hw32, int col_tiles, int n_items) {
  pdl_launch_dependents();
  using C = BMCfg<CW>;
  extern __shared__ __align__(128) uint8_t smem[];
  uint2* lut = reinterpret_cast<uint2*>(smem);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int e = threadIdx.x; e < 1024; e += BM_THREADS) lut[e] = lut_entry_masked(e & 63u, e >> 6, N);
  pdl_wait();                                              // the table needed no global memory
  __syncthreads();
  const int nw = gridDim.x * BM_WARPS;
  int item = blockIdx.x * BM_WARPS + warp;
  if (item >= n_items) return;
  uint8_t* my_ring = smem + C::LUT_BYTES + warp * BM_RING * C::STAGE;
  const uint32_t ring_u32 = ptx::smem_u32(my_ring);
  const int jwords = J >> 5;
  const unsigned last_row = (unsigned)(I - 1);
  const int step_rg = nw / col_tiles, step_ct = nw % col_tiles;
  int rg = item / col_tiles, ct = item % col_tiles;        // 32-row group and column tile of the item

  // the gather of row-block j of an item whose 32 row indices the lanes hold in `rows`
  auto issue = [&](int rows, int ctile, int j) {
    const uint32_t dst = ring_u32 + (j % BM_RING) * C::STAGE;
    // a row slice is 128 CW bytes = 8 CW lanes x 16 bytes: CW passes of 4 / CW rows each
#pragma unroll
    for (int ps = 0; ps < CW; ++ps) {
      const int m = ps * (4 / CW) + lane / (8 * CW), piece = lane % (8 * CW);
      const int r = __shfl_sync(0xFFFFFFFFu, rows, 4 * j + m);
      cp_async16(dst + m * 128 * CW + 16 * piece, W + (size_t)r * J + ctile * 32 * CW + 4 * piece);
    }
    cp_async_commit();
  };
  auto load_rows = [&](int rgroup) { return (int)min((unsigned)__ldg(perm + 32 * rgroup + lane), last_row); };
  auto load_fwd = [&](int rows, int ctile, uint32_t (&f)[CW]) {
    const uint32_t* src = maskbits_f + (size_t)rows * jwords + ctile * CW;
    if (CW == 2) { const uint2 t = __ldg(reinterpret_cast<const uint2*>(src)); f[0] = t.x; f[1] = t.y; }
    else f[0] = __ldg(src);
  };

  int rows_nxt = load_rows(rg);
  uint32_t f_nxt[CW];
  load_fwd(rows_nxt, ct, f_nxt);
  issue(rows_nxt, ct, 0);
  issue(rows_nxt, ct, 1);
  issue(rows_nxt, ct, 2);
  const size_t vrow = (size_t)I >> 2;                      // u32 (bf16 pairs) per row of vals_b
  const size_t mrow = (size_t)I >> 5;
  while (true) {
    const int rows_cur = rows_nxt;
    uint32_t cand[CW];                                     // candidate bits of this lane's columns, by row
#pragma unroll
    for (int c = 0; c < CW; ++c) cand[c] = transpose32(f_nxt[c], lane);
    int rg_n = rg + step_rg, ct_n = ct + step_ct;
    if (ct_n >= col_tiles) { ct_n -= col_tiles; ++rg_n; }
    const bool has_next = item + nw < n_items;             // warp uniform
    if (has_next) rows_nxt = load_rows(rg_n);
    uint32_t vacc[CW][8];
    uint32_t cacc[CW], kacc[CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) cacc[c] = kacc[c] = 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (j + 3 < 8) issue(rows_cur, ct, j + 3);
      else if (has_next) issue(rows_nxt, ct_n, j + 3 - 8);  // the ring runs on into the next item
      else cp_async_commit();                              // keep the group count uniform
      if (j == 4 && has_next) load_fwd(rows_nxt, ct_n, f_nxt);
      cp_async_wait<3>();                                  // row-block j has landed
      __syncwarp();
      const float* ws = reinterpret_cast<const float*>(my_ring + (j % BM_RING) * C::STAGE);
      float w[4][CW];
#pragma unroll
      for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int c = 0; c < CW; ++c) w[m][c] = ws[m * 32 * CW + 32 * c + lane];
      __syncwarp();                                        // all lanes have read the stage
#pragma unroll
      for (int c = 0; c < CW; ++c) {
        const uint32_t k0 = mag_key(w[0][c]), k1 = mag_key(w[1][c]), k2 = mag_key(w[2][c]), k3 = mag_key(w[3][c]);
        const uint32_t valid = (cand[c] >> (4 * j)) & 15u;
        const uint2 e = lut[(valid << 6) | cmp6(k0, k1, k2, k3)];
        vacc[c][j] = slots_masked(e, w[0][c], w[1][c], w[2][c], w[3][c], k0, k1, k2, k3);
        kacc[c] |= ((e.x >> 16) & 15u) << (4 * j);
        cacc[c] |= ((e.x >> 20) & 15u) << (4 * j);
      }
    }
    // this warp's 32 permuted rows of backward-mask words: one store of CW words per lane
    uint32_t* mrow_out = maskbits_b + (size_t)(32 * rg + lane) * jwords + ct * CW;
    if (CW == 2) *reinterpret_cast<uint2*>(mrow_out) = make_uint2(transpose32(kacc[0], lane), transpose32(kacc[1], lane));
    else *mrow_out = transpose32(kacc[0], lane);
#pragma unroll
    for (int c = 0; c < CW; ++c) {
      const int l = (ct * CW + c) * 32 + lane;
      uint4* dst = reinterpret_cast<uint4*>(vals_b + (size_t)l * vrow + 8 * rg);
      dst[0] = make_uint4(vacc[c][0], vacc[c][1], vacc[c][2], vacc[c][3]);
      dst[1] = make_uint4(vacc[c][4], vacc[c][5], vacc[c][6], vacc[c][7]);
      meta_b[(size_t)l * mrow + rg] = cacc[c];
      if (hw32) {
        // image word (rows l and l ^ 8 of the operand, k word rg): its low-half lane stores the two low halves of
        // the code words, its high-half lane the two high halves
        const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, cacc[c], 8);
        const int rr = l & 127;
        const size_t tile = (size_t)(l >> 7) * (I >> 7) + (rg >> 2);
        const size_t at = tile * 512 + (size_t)((rr & 7) + 16 * (rr >> 4)) * 4 + (rg & 3);
        if (rr & 8) hw32[at + 32] = __byte_perm(other, cacc[c], 0x7632u);
        else hw32[at] = __byte_perm(cacc[c], other, 0x5410u);
      }
    }
    if (!has_next) break;
    item += nw;
    rg = rg_n;
    ct = ct_n;
  }
  cp_async_wait<0>();
}

}  // namespace

int launch_fwd_mask(const float* W, int I, int J, int N, uint32_t* maskbits, uint16_t* vals,
                    uint32_t* meta, void* hw_meta_or_null, cudaStream_t s) {
  uint16_t* hw16 = reinterpret_cast<uint16_t*>(hw_meta_or_null);
  const long long nblk = (long long)I * J / 4;
  const long long nchunks = (nblk + 255) >> 8;
  long long ctas = (nchunks + 7) / 8;
  if (ctas > 148 * 8) ctas = 148 * 8;
  if (ctas < 1) ctas = 1;
  const SgdParams none{nullptr, nullptr, nullptr, 0.f, 0.f, 0.f};
  if (N == 2)
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<true, false>, (unsigned)ctas, FWD_THREADS, 0, s,
        reinterpret_cast<const float4*>(W), nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, none));
  else
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<false, false>, (unsigned)ctas, FWD_THREADS, 0, s,
        reinterpret_cast<const float4*>(W), nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, none));
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
  if (N == 2)
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<true, true>, (unsigned)ctas, FWD_THREADS, 0, s,
        nullptr, nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, p));
  else
    BIMASK_CUDA_OK(launch_pdl(fwd_mask_pack_kernel<false, true>, (unsigned)ctas, FWD_THREADS, 0, s,
        nullptr, nblk, N, maskbits, reinterpret_cast<uint4*>(vals), meta, hw16, J / 32, p));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// Plain update pass (same arithmetic), for the patterns whose mask kernel is the generic one.
__global__ void sgd_update_kernel(long long n4, SgdParams p) {
  pdl_launch_dependents();
  pdl_wait();
  for (long long at = (long long)blockIdx.x * blockDim.x + threadIdx.x; at < n4; at += (long long)gridDim.x * blockDim.x) {
    float4 w = p.W4[at];
    const float4 dw = __ldg(p.dW4 + at);
    float4 m = p.mom4 ? p.mom4[at] : make_float4(0.f, 0.f, 0.f, 0.f);
    w.x = sgd_one(w.x, dw.x, m.x, p);
    w.y = sgd_one(w.y, dw.y, m.y, p);
    w.z = sgd_one(w.z, dw.z, m.z, p);
    w.w = sgd_one(w.w, dw.w, m.w, p);
    p.W4[at] = w;
    if (p.mom4) p.mom4[at] = m;
  }
}

int launch_sgd_update(float* W, const float* dW, float* mom, long long n, float lr, float momentum, float weight_decay,
                      cudaStream_t s) {
  const long long n4 = n / 4;
  long long ctas = (n4 + 255) / 256;
  if (ctas > 148 * 8) ctas = 148 * 8;
  if (ctas < 1) ctas = 1;
  const SgdParams p{reinterpret_cast<float4*>(W), reinterpret_cast<const float4*>(dW), reinterpret_cast<float4*>(mom),
                    lr, momentum, weight_decay};
  BIMASK_CUDA_OK(launch_pdl(sgd_update_kernel, (unsigned)ctas, 256, 0, s, n4, p));
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
  // 64-column items once they keep every resident warp busy, 32-column items (twice as many) otherwise
  const long long items_wide = (long long)(I / 32) * (J / 64);
  const bool wide = J % 64 == 0 && items_wide >= (long long)BM_CTAS_PER_SM * 148 * BM_WARPS;
  const int col_tiles = wide ? J / 64 : J / 32;
  const long long n_items = (long long)(I / 32) * col_tiles;
  BIMASK_REQUIRE(n_items < (1ll << 31), BIMASK_EUNSUPPORTED, "bimask_bwd_mask: I * J = %lld is beyond the kernel's item index",
                 (long long)I * J);
  long long ctas = (n_items + BM_WARPS - 1) / BM_WARPS;
  if (ctas > BM_CTAS_PER_SM * 148) ctas = BM_CTAS_PER_SM * 148;
  uint32_t* vals32 = reinterpret_cast<uint32_t*>(vals_b);
  uint32_t* hw32 = reinterpret_cast<uint32_t*>(hw_meta_or_null);
  if (wide) {
    if (int rc = set_smem_attr(bwd_mask_kernel<2>, BMCfg<2>::SMEM)) return rc;
    BIMASK_CUDA_OK(launch_pdl(bwd_mask_kernel<2>, (unsigned)ctas, BM_THREADS, BMCfg<2>::SMEM, s, W, maskbits_f, perm, I, J, N,
                              maskbits_b, vals32, meta_b, hw32, col_tiles, (int)n_items));
  } else {
    if (int rc = set_smem_attr(bwd_mask_kernel<1>, BMCfg<1>::SMEM)) return rc;
    BIMASK_CUDA_OK(launch_pdl(bwd_mask_kernel<1>, (unsigned)ctas, BM_THREADS, BMCfg<1>::SMEM, s, W, maskbits_f, perm, I, J, N,
                              maskbits_b, vals32, meta_b, hw32, col_tiles, (int)n_items));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace bimask
