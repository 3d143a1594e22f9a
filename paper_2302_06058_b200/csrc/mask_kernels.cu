// Forward mask + 2:4 packing (Eq. 4), backward mask + transposed packing (Eq. 11) and the
// re-ordering of the index metadata into the tensor core's TMEM image.
//
// All three are streaming kernels bound by HBM: every weight is read once per kernel with
// coalesced 128-bit (forward) or 128-byte-per-warp (backward, row gather) accesses, the
// selection is done on integer magnitude keys in registers, and the bit/nibble words are
// assembled with warp reductions / ballots so that every store is a full word.
#include "common.cuh"

namespace bimask {

namespace {

__device__ __forceinline__ uint32_t mag_key(float w) { return __float_as_uint(w) & 0x7FFFFFFFu; }

// fp32 -> bf16, round to nearest even; NaN -> quiet NaN keeping sign and top payload bits.
__device__ __forceinline__ uint32_t to_bf16(float w) {
  uint32_t u = __float_as_uint(w);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 16) | 0x40u;
  return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

// Rank selection inside one block of four: element m is kept when it is a candidate
// (bit m of `valid`) and fewer than N candidates beat it; q beats m when key_q > key_m, or
// key_q == key_m with q < m.  Returns the 4-bit keep mask.
__device__ __forceinline__ uint32_t keep4(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3,
                                          uint32_t valid, int N) {
  const uint32_t v0 = valid & 1u, v1 = (valid >> 1) & 1u, v2 = (valid >> 2) & 1u, v3 = (valid >> 3) & 1u;
  // b_qm = 1 when the lower-index element q beats the higher-index element m (ties -> q)
  const uint32_t b01 = k0 >= k1, b02 = k0 >= k2, b03 = k0 >= k3;
  const uint32_t b12 = k1 >= k2, b13 = k1 >= k3, b23 = k2 >= k3;
  const uint32_t r0 = (v1 & (b01 ^ 1u)) + (v2 & (b02 ^ 1u)) + (v3 & (b03 ^ 1u));
  const uint32_t r1 = (v0 & b01) + (v2 & (b12 ^ 1u)) + (v3 & (b13 ^ 1u));
  const uint32_t r2 = (v0 & b02) + (v1 & b12) + (v3 & (b23 ^ 1u));
  const uint32_t r3 = (v0 & b03) + (v1 & b13) + (v2 & b23);
  const uint32_t n = (uint32_t)N;
  return (v0 & (r0 < n)) | ((v1 & (r1 < n)) << 1) | ((v2 & (r2 < n)) << 2) | ((v3 & (r3 < n)) << 3);
}

// 2:4 container for a block with at most two kept elements: index code and the two bf16 slots.
__device__ __forceinline__ void pack4(uint32_t kb, float w0, float w1, float w2, float w3,
                                      uint32_t& code, uint32_t& vals) {
  const int pop = __popc(kb);
  const uint32_t lo = (uint32_t)(__ffs(kb) - 1);          // lowest kept (unused if pop == 0)
  uint32_t idx0, idx1;
  if (pop >= 2) {
    idx0 = lo;
    idx1 = 31u - (uint32_t)__clz(kb);
  } else if (pop == 1) {
    idx0 = 0u;
    idx1 = lo < 1u ? 1u : lo;
  } else {
    idx0 = 0u;
    idx1 = 1u;
  }
  const float s0 = idx0 == 0 ? w0 : idx0 == 1 ? w1 : idx0 == 2 ? w2 : w3;
  const float s1 = idx1 == 0 ? w0 : idx1 == 1 ? w1 : idx1 == 2 ? w2 : w3;
  const uint32_t a = ((kb >> idx0) & 1u) ? to_bf16(s0) : 0u;
  const uint32_t b = ((kb >> idx1) & 1u) ? to_bf16(s1) : 0u;
  code = idx0 | (idx1 << 2);
  vals = a | (b << 16);
}

// ---------------------------------------------------------------------------------------
// Forward mask + pack.  W is treated as a flat stream of 4-element blocks (J % 32 == 0, so
// blocks, 32-column words and rows all nest).  A warp owns chunks of 256 blocks: 8 coalesced
// float4 loads per lane are issued up front, then each lane's 4 mask bits / index nibble are
// OR-reduced over 8-lane groups into words and routed so that lane w stores word w of the
// chunk (one coalesced 128-byte store each for maskbits and meta).
// ---------------------------------------------------------------------------------------
constexpr int FWD_THREADS = 256;

__global__ void __launch_bounds__(FWD_THREADS)
fwd_mask_pack_kernel(const float4* __restrict__ W4, long long nblk, int N,
                     uint32_t* __restrict__ maskbits, uint32_t* __restrict__ vals,
                     uint32_t* __restrict__ meta) {
  const int lane = threadIdx.x & 31;
  const long long warp = ((long long)blockIdx.x * FWD_THREADS + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * FWD_THREADS) >> 5;
  const long long nchunks = (nblk + 255) >> 8;
  const uint32_t gmask = 0xFFu << (lane & 24);
  const int sh = 4 * (lane & 7);
  for (long long ch = warp; ch < nchunks; ch += nwarps) {
    const long long base = ch << 8;
    float4 w[8];
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const long long b = base + it * 32 + lane;
      w[it] = b < nblk ? __ldg(W4 + b) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    uint32_t my_bits = 0, my_meta = 0;
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const long long b = base + it * 32 + lane;
      const uint32_t kb = keep4(mag_key(w[it].x), mag_key(w[it].y), mag_key(w[it].z), mag_key(w[it].w), 0xFu, N);
      uint32_t code, v;
      pack4(kb, w[it].x, w[it].y, w[it].z, w[it].w, code, v);
      if (b < nblk) vals[b] = v;
      const uint32_t wb = __reduce_or_sync(gmask, kb << sh);
      const uint32_t wm = __reduce_or_sync(gmask, code << sh);
      const uint32_t rb = __shfl_sync(0xFFFFFFFFu, wb, (lane & 3) * 8);
      const uint32_t rm = __shfl_sync(0xFFFFFFFFu, wm, (lane & 3) * 8);
      if ((lane >> 2) == it) { my_bits = rb; my_meta = rm; }
    }
    const long long word = (base >> 3) + lane;
    if (word < (nblk >> 3)) {
      maskbits[word] = my_bits;
      meta[word] = my_meta;
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
                               int tiles_k, long long total, uint32_t* __restrict__ out) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= total) return;
  const int c = (int)(idx & 3);
  const int L = (int)((idx >> 2) & 127);
  const long long tile = idx >> 9;
  const int kt = (int)(tile % tiles_k);
  const int mt = (int)(tile / tiles_k);
  const int m0 = L & 7, h = (L >> 3) & 1, m2 = L >> 4;
  const int r_lo = mt * 128 + m0 + 16 * m2;
  const int r_hi = r_lo + 8;
  const int w = kt * 4 + c;
  uint32_t lo = 0x4444u, hi = 0x4444u;
  if (w < kwords) {
    if (r_lo < rows) lo = (__ldg(meta + (long long)r_lo * kwords + w) >> (16 * h)) & 0xFFFFu;
    if (r_hi < rows) hi = (__ldg(meta + (long long)r_hi * kwords + w) >> (16 * h)) & 0xFFFFu;
  }
  out[idx] = lo | (hi << 16);
}

// ---------------------------------------------------------------------------------------
// Backward mask + transposed pack.  A CTA owns 128 columns x 64 row-blocks (256 permuted
// rows).  Warp w handles row-blocks w, w+8, ...: for a row-block it gathers the four source
// rows perm[4k..4k+3]; lane handles columns lane + 32 q (q < 4) so every load is a coalesced
// 128-byte segment and a ballot over the warp yields a complete mask word.  The (value pair,
// index code) of block (k, l) belongs to row l of the transposed operand, so it is staged in
// shared memory ([l][k], padded) and written out with k contiguous.
// ---------------------------------------------------------------------------------------
constexpr int BWD_COLS = 128;
constexpr int BWD_KB = 64;
constexpr int BWD_THREADS = 256;
constexpr int BWD_VSTRIDE = BWD_KB + 1;   // u32 words per staged row (odd => conflict-free)
constexpr int BWD_CSTRIDE = BWD_KB + 4;   // bytes per staged code row (17 words, odd)

__global__ void __launch_bounds__(BWD_THREADS)
bwd_mask_pack_kernel(const float* __restrict__ W, const uint32_t* __restrict__ maskbits_f,
                     const int32_t* __restrict__ perm, int I, int J, int N,
                     uint32_t* __restrict__ maskbits_b, uint32_t* __restrict__ vals_b,
                     uint32_t* __restrict__ meta_b) {
  __shared__ uint32_t vals_s[BWD_COLS * BWD_VSTRIDE];
  __shared__ uint8_t code_s[BWD_COLS * BWD_CSTRIDE];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col0 = blockIdx.x * BWD_COLS;
  const int kb0 = blockIdx.y * BWD_KB;
  const int nkb = I >> 2;
  const int jwords = J >> 5;
  const int kb_here = min(BWD_KB, nkb - kb0);
  const int cols_here = min(BWD_COLS, J - col0);          // multiple of 32
  const int nq = cols_here >> 5;

  for (int kk = warp; kk < kb_here; kk += BWD_THREADS / 32) {
    const int k = kb0 + kk;
    const int4 p4 = __ldg(reinterpret_cast<const int4*>(perm) + k);
    const int src[4] = {p4.x, p4.y, p4.z, p4.w};
    float w[4][4];
    uint32_t fb[4][4];
#pragma unroll
    for (int m = 0; m < 4; ++m)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (q < nq) {
          w[m][q] = __ldg(W + (long long)src[m] * J + col0 + 32 * q + lane);
          fb[m][q] = __ldg(maskbits_f + (long long)src[m] * jwords + (col0 >> 5) + q);
        } else {
          w[m][q] = 0.f;
          fb[m][q] = 0u;
        }
      }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (q >= nq) break;
      const uint32_t valid = ((fb[0][q] >> lane) & 1u) | (((fb[1][q] >> lane) & 1u) << 1) |
                             (((fb[2][q] >> lane) & 1u) << 2) | (((fb[3][q] >> lane) & 1u) << 3);
      const uint32_t kb = keep4(mag_key(w[0][q]), mag_key(w[1][q]), mag_key(w[2][q]), mag_key(w[3][q]), valid, N);
      uint32_t code, v;
      pack4(kb, w[0][q], w[1][q], w[2][q], w[3][q], code, v);
      const int l = 32 * q + lane;
      vals_s[l * BWD_VSTRIDE + kk] = v;
      code_s[l * BWD_CSTRIDE + kk] = (uint8_t)code;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const uint32_t word = __ballot_sync(0xFFFFFFFFu, (kb >> m) & 1u);
        if (lane == m) maskbits_b[(long long)(4 * k + m) * jwords + (col0 >> 5) + q] = word;
      }
    }
  }
  __syncthreads();
  // transposed operand: row l = column of W, k contiguous
  const long long vrow = (long long)(I >> 1) >> 1;     // u32 (bf16 pairs) per row of vals_b = I/4
  for (int l = warp; l < cols_here; l += BWD_THREADS / 32) {
    for (int kk = lane; kk < kb_here; kk += 32)
      vals_b[(long long)(col0 + l) * vrow + kb0 + kk] = vals_s[l * BWD_VSTRIDE + kk];
  }
  const int mwords_here = kb_here >> 3;                // I % 32 == 0 => whole words
  const int mrow = I >> 5;
  for (int e = threadIdx.x; e < cols_here * mwords_here; e += BWD_THREADS) {
    const int l = e / mwords_here, wd = e % mwords_here;
    uint32_t word = 0;
#pragma unroll
    for (int g = 0; g < 8; ++g) word |= (uint32_t)code_s[l * BWD_CSTRIDE + 8 * wd + g] << (4 * g);
    meta_b[(long long)(col0 + l) * mrow + (kb0 >> 3) + wd] = word;
  }
}

}  // namespace

int launch_fwd_mask(const float* W, int I, int J, int N, uint32_t* maskbits, uint16_t* vals,
                    uint32_t* meta, cudaStream_t s) {
  const long long nblk = (long long)I * J / 4;
  const long long nchunks = (nblk + 255) >> 8;
  long long ctas = (nchunks + 7) / 8;
  if (ctas > 148 * 8) ctas = 148 * 8;
  if (ctas < 1) ctas = 1;
  fwd_mask_pack_kernel<<<(unsigned)ctas, FWD_THREADS, 0, s>>>(
      reinterpret_cast<const float4*>(W), nblk, N, maskbits, reinterpret_cast<uint32_t*>(vals), meta);
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_hw_meta(const uint32_t* meta, int rows, int K, void* hw_meta, cudaStream_t s) {
  const int tiles_m = (rows + 127) / 128, tiles_k = (K + 127) / 128;
  const long long total = (long long)tiles_m * tiles_k * 512;
  hw_meta_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(meta, rows, K / 32, tiles_k, total,
                                                                 reinterpret_cast<uint32_t*>(hw_meta));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_bwd_mask(const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                    int N, uint32_t* maskbits_b, uint16_t* vals_b, uint32_t* meta_b, cudaStream_t s) {
  dim3 grid((J + BWD_COLS - 1) / BWD_COLS, (I / 4 + BWD_KB - 1) / BWD_KB);
  bwd_mask_pack_kernel<<<grid, BWD_THREADS, 0, s>>>(W, maskbits_f, perm, I, J, N, maskbits_b,
                                                    reinterpret_cast<uint32_t*>(vals_b), meta_b);
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace bimask
