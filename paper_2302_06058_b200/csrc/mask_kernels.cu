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
// Backward mask + transposed pack, asynchronous-copy variant.  A CTA owns 32 CW columns x 64 row-blocks (256
// permuted rows); warp w walks the eight consecutive row-blocks 8w .. 8w+7.  Each warp runs its own three-deep
// ring of shared-memory stages filled with cp.async (the slices of the four gathered rows plus their forward-mask
// words), so the gather of row-block j+2 is in flight while row-block j is processed and costs no registers.
// Compute uses lane = column within each of the tile's CW 32-column words: conflict-free shared loads, and a warp
// ballot yields a complete backward-mask word.  The operand being produced is transposed (row = column l of W,
// k contiguous): each lane keeps the eight consecutive k results of its CW columns in registers and writes them
// as full 32-byte sectors.
// CW = 2 (J a multiple of 64) is the variant for large matrices: 256-byte row slices, 64 registers, four CTAs
// per SM (CW = 4 needs 80 registers, runs three and measured 4 % slower).
// CW = 1 has twice as many warps again for the same matrix; it serves small matrices, where the per-warp chain
// of eight row-blocks is what takes the time, and any J % 32 == 0.
// ---------------------------------------------------------------------------------------
constexpr int B4_KB = 64, B4_WARPS = 8, B4_THREADS = 32 * B4_WARPS, B4_RING = 3;
template <int CW>
struct B4Cfg {
  static constexpr int STAGE = 4 * 128 * CW + 64;          // four row slices + four x 16 bytes for the mask words
  static constexpr int SMEM = B4_WARPS * B4_RING * STAGE + 4 * B4_KB * 16 + 1024 * 4 + B4_KB * 16;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
template <int WORDS>                                       // 1, 2 or 4 32-bit words
__device__ __forceinline__ void cp_async_words(uint32_t dst, const void* src) {
  if (WORDS == 4) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
  else if (WORDS == 2) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
  else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int CW>
__global__ void __launch_bounds__(B4_THREADS, 4)
bwd_mask_async_kernel(const float* __restrict__ W, const uint32_t* __restrict__ maskbits_f,
                      const int32_t* __restrict__ perm, int I, int J, int N,
                      uint32_t* __restrict__ maskbits_b, uint32_t* __restrict__ vals_b,
                      uint32_t* __restrict__ meta_b, uint16_t* __restrict__ hw16) {
  pdl_launch_dependents();
  using C = B4Cfg<CW>;
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* ring = smem;                                                          // [warp][stage][C::STAGE]
  uint4* mb_s = reinterpret_cast<uint4*>(smem + B4_WARPS * B4_RING * C::STAGE);  // [256 rows] x up to 4 mask words
  uint32_t* lut = reinterpret_cast<uint32_t*>(mb_s + 4 * B4_KB);                 // [1024]
  int4* perm_s = reinterpret_cast<int4*>(lut + 1024);                            // [64]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = blockIdx.y * 32 * CW;                   // J % (32 CW) == 0: the tile is always full
  const int kb0 = blockIdx.x * B4_KB;
  const int kb_here = min(B4_KB, (I >> 2) - kb0);          // multiple of 8 (I % 32 == 0)
  const int jwords = J >> 5;
  const unsigned last_row = (unsigned)(I - 1);

  for (int e = threadIdx.x; e < 1024; e += B4_THREADS) lut[e] = lut_entry(e & 63u, e >> 6, N);
  pdl_wait();                                              // the table needed no global memory
  for (int kk = threadIdx.x; kk < kb_here; kk += B4_THREADS) {
    const int4 p4 = __ldg(reinterpret_cast<const int4*>(perm) + kb0 + kk);
    perm_s[kk] = make_int4((int)min((unsigned)p4.x, last_row), (int)min((unsigned)p4.y, last_row),
                           (int)min((unsigned)p4.z, last_row), (int)min((unsigned)p4.w, last_row));
  }
  __syncthreads();
  const int kw = 8 * warp;                                 // this warp's row-blocks kw .. kw+7 of the tile
  if (kw < kb_here) {
    uint8_t* my_ring = ring + warp * B4_RING * C::STAGE;
    const uint32_t ring_u32 = ptx::smem_u32(my_ring);
    auto issue = [&](int j) {                              // start the gather of row-block kw + j
      const int4 p4 = perm_s[kw + j];
      const int r[4] = {p4.x, p4.y, p4.z, p4.w};
      const uint32_t dst = ring_u32 + (j % B4_RING) * C::STAGE;
      // a row slice is 128 CW bytes = 8 CW lanes x 16 bytes: CW passes of 4 / CW rows each
#pragma unroll
      for (int ps = 0; ps < CW; ++ps) {
        const int m = ps * (4 / CW) + lane / (8 * CW), piece = lane % (8 * CW);
        cp_async16(dst + m * 128 * CW + 16 * piece, W + (size_t)r[m] * J + col0 + 4 * piece);
      }
      if (lane < 4) cp_async_words<CW>(dst + 512 * CW + 16 * lane, maskbits_f + (size_t)r[lane] * jwords + (col0 >> 5));
      cp_async_commit();
    };
    issue(0);
    issue(1);
    uint32_t vacc[CW][8];
    uint32_t cacc[CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) cacc[c] = 0u;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (j + 2 < 8) issue(j + 2); else cp_async_commit();  // keep the group count uniform
      cp_async_wait<2>();                                  // row-block j has landed
      __syncwarp();
      const float* ws = reinterpret_cast<const float*>(my_ring + (j % B4_RING) * C::STAGE);
      const uint4* fs = reinterpret_cast<const uint4*>(my_ring + (j % B4_RING) * C::STAGE + 128 * CW * 4);
      float w[4][CW];
      uint4 fw[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        if (CW == 4) fw[m] = fs[m];
        else if (CW == 2) { const uint2 t = reinterpret_cast<const uint2*>(fs + m)[0]; fw[m].x = t.x; fw[m].y = t.y; }
        else fw[m].x = reinterpret_cast<const uint32_t*>(fs + m)[0];
#pragma unroll
        for (int c = 0; c < CW; ++c) w[m][c] = ws[m * 32 * CW + 32 * c + lane];
      }
      __syncwarp();                                        // all lanes have read the stage
      const int kk = kw + j;
#pragma unroll
      for (int c = 0; c < CW; ++c) {
        const uint32_t f0 = c == 0 ? fw[0].x : c == 1 ? fw[0].y : c == 2 ? fw[0].z : fw[0].w;
        const uint32_t f1 = c == 0 ? fw[1].x : c == 1 ? fw[1].y : c == 2 ? fw[1].z : fw[1].w;
        const uint32_t f2 = c == 0 ? fw[2].x : c == 1 ? fw[2].y : c == 2 ? fw[2].z : fw[2].w;
        const uint32_t f3 = c == 0 ? fw[3].x : c == 1 ? fw[3].y : c == 2 ? fw[3].z : fw[3].w;
        const uint32_t valid = ((f0 >> lane) & 1u) | (((f1 >> lane) & 1u) << 1) | (((f2 >> lane) & 1u) << 2) |
                               (((f3 >> lane) & 1u) << 3);
        const uint32_t k0 = mag_key(w[0][c]), k1 = mag_key(w[1][c]), k2 = mag_key(w[2][c]), k3 = mag_key(w[3][c]);
        const uint32_t e = lut[(valid << 6) | cmp6(k0, k1, k2, k3)];
        vacc[c][j] = slots<false>(e, w[0][c], w[1][c], w[2][c], w[3][c], k0, k1, k2, k3);
        cacc[c] |= ((e >> 4) & 15u) << (4 * j);
        uint32_t b[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) b[m] = __ballot_sync(0xFFFFFFFFu, (e >> m) & 1u);
        if (lane == 0) {
#pragma unroll
          for (int m = 0; m < 4; ++m) reinterpret_cast<uint32_t*>(mb_s + 4 * kk + m)[c] = b[m];
        }
      }
    }
    cp_async_wait<0>();
    __syncwarp();
    // this warp's 32 permuted rows of backward-mask words: one store of CW words per lane
    uint32_t* mrow_out = maskbits_b + (size_t)(4 * (kb0 + kw) + lane) * jwords + (col0 >> 5);
    if (CW == 4) *reinterpret_cast<uint4*>(mrow_out) = mb_s[4 * kw + lane];
    else if (CW == 2) *reinterpret_cast<uint2*>(mrow_out) = reinterpret_cast<const uint2*>(mb_s + 4 * kw + lane)[0];
    else *mrow_out = reinterpret_cast<const uint32_t*>(mb_s + 4 * kw + lane)[0];
    const size_t vrow = (size_t)I >> 2;                    // u32 (bf16 pairs) per row of vals_b
    const size_t mrow = (size_t)I >> 5;
#pragma unroll
    for (int c = 0; c < CW; ++c) {
      const int l = col0 + 32 * c + lane;
      uint4* dst = reinterpret_cast<uint4*>(vals_b + (size_t)l * vrow + kb0 + kw);
      dst[0] = make_uint4(vacc[c][0], vacc[c][1], vacc[c][2], vacc[c][3]);
      dst[1] = make_uint4(vacc[c][4], vacc[c][5], vacc[c][6], vacc[c][7]);
      meta_b[(size_t)l * mrow + ((kb0 + kw) >> 3)] = cacc[c];
      if (hw16) scatter_hw(hw16, I >> 7, l, (kb0 + kw) >> 3, cacc[c]);
    }
  }
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
  // the wide tile (64 columns per warp) once it gives every SM a few CTAs, the narrow one otherwise
  const int row_tiles = (I / 4 + B4_KB - 1) / B4_KB;
  const bool wide = J % 64 == 0 && (long long)row_tiles * (J / 64) >= 4 * 148;
  static bool attr_done = false;
  if (!attr_done) {
    BIMASK_CUDA_OK(cudaFuncSetAttribute(bwd_mask_async_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, B4Cfg<2>::SMEM));
    BIMASK_CUDA_OK(cudaFuncSetAttribute(bwd_mask_async_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, B4Cfg<1>::SMEM));
    attr_done = true;
  }
  uint32_t* vals32 = reinterpret_cast<uint32_t*>(vals_b);
  uint16_t* hw16 = reinterpret_cast<uint16_t*>(hw_meta_or_null);
  if (wide) {
    dim3 grid(row_tiles, J / 64);
    BIMASK_CUDA_OK(launch_pdl(bwd_mask_async_kernel<2>, grid, B4_THREADS, B4Cfg<2>::SMEM, s, W, maskbits_f, perm, I, J, N, maskbits_b, vals32, meta_b, hw16));
  } else {
    dim3 grid(row_tiles, J / 32);
    BIMASK_CUDA_OK(launch_pdl(bwd_mask_async_kernel<1>, grid, B4_THREADS, B4Cfg<1>::SMEM, s, W, maskbits_f, perm, I, J, N, maskbits_b, vals32, meta_b, hw16));
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace bimask
