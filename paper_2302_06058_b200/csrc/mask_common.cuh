// Device helpers shared by the mask kernels: magnitude keys, bf16 rounding, and the table-driven
// selection inside one group of four.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bimask {
namespace {

__device__ __forceinline__ uint32_t mag_key(float w) { return __float_as_uint(w) & 0x7FFFFFFFu; }

// fp32 -> bf16, round to nearest even; NaN -> quiet NaN keeping sign and top payload bits.
__device__ __forceinline__ uint32_t to_bf16(float w) {
  uint32_t u = __float_as_uint(w);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 16) | 0x40u;
  return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

// Selection inside one block of four, table driven.  The six pairwise magnitude comparisons
// (b_qm = key_q >= key_m for q < m) and the four candidate bits index a table whose entry holds
// everything the block needs:
//   bits [0,4)   keep mask: element m is kept when it is a candidate and fewer than N candidates
//                beat it; q beats m when key_q > key_m, or key_q == key_m with q < m
//   bits [4,8)   index code idx0 | idx1 << 2 of the 2:4 container (pad rule for < 2 kept)
//   bit 8 / 9    slot 0 / slot 1 holds a kept element (else the slot is +0)
//   bits [16,32) byte-permute selector that picks the two slots out of the four bf16 values
// The table (64 entries for "all candidates", 1024 with candidate bits) is rebuilt in shared
// memory by every CTA from the rule itself.
__device__ __forceinline__ uint32_t lut_entry(uint32_t cmp, uint32_t valid, int N) {
  const uint32_t b01 = (cmp >> 5) & 1u, b02 = (cmp >> 4) & 1u, b03 = (cmp >> 3) & 1u;
  const uint32_t b12 = (cmp >> 2) & 1u, b13 = (cmp >> 1) & 1u, b23 = cmp & 1u;
  const uint32_t v0 = valid & 1u, v1 = (valid >> 1) & 1u, v2 = (valid >> 2) & 1u, v3 = (valid >> 3) & 1u;
  const uint32_t r0 = (v1 & (b01 ^ 1u)) + (v2 & (b02 ^ 1u)) + (v3 & (b03 ^ 1u));
  const uint32_t r1 = (v0 & b01) + (v2 & (b12 ^ 1u)) + (v3 & (b13 ^ 1u));
  const uint32_t r2 = (v0 & b02) + (v1 & b12) + (v3 & (b23 ^ 1u));
  const uint32_t r3 = (v0 & b03) + (v1 & b13) + (v2 & b23);
  const uint32_t n = (uint32_t)N;
  const uint32_t kb = (v0 & (r0 < n)) | ((v1 & (r1 < n)) << 1) | ((v2 & (r2 < n)) << 2) | ((v3 & (r3 < n)) << 3);
  const int pop = __popc(kb);
  uint32_t idx0 = 0u, idx1 = 1u;
  if (pop >= 2) {
    idx0 = (uint32_t)(__ffs(kb) - 1);
    idx1 = 31u - (uint32_t)__clz(kb);
  } else if (pop == 1) {
    const uint32_t lo = (uint32_t)(__ffs(kb) - 1);
    idx1 = lo < 1u ? 1u : lo;
  }
  const uint32_t sel = (2u * idx0) | ((2u * idx0 + 1u) << 4) | ((2u * idx1) << 8) | ((2u * idx1 + 1u) << 12);
  return kb | (idx0 << 4) | (idx1 << 6) | (((kb >> idx0) & 1u) << 8) | (((kb >> idx1) & 1u) << 9) | (sel << 16);
}

// The same entry laid out for the backward-mask kernel:
//   bits [0,16)  byte-permute selector of the two slots (the permute reads its low 16 bits in place)
//   bits [16,20) keep mask, bits [24,28) index code
//   bit 31 / 23  slot 0 / slot 1 holds a kept element: the top bits of bytes 3 and 2, so that one byte permute in
//                sign-replication mode expands them into the 0xFFFF / 0 halves of the slot mask
__device__ __forceinline__ uint32_t lut_entry_signs(uint32_t cmp, uint32_t valid, int N) {
  const uint32_t e = lut_entry(cmp, valid, N);
  return (e >> 16) | ((e & 0xFu) << 16) | (((e >> 4) & 0xFu) << 24) | (((e >> 8) & 1u) << 31) | (((e >> 9) & 1u) << 23);
}

// Six comparison bits of a block, b01 first (bit 5) ... b23 last (bit 0).  Keys are < 2^31, so
// key_m - key_q - 1 is negative exactly when key_q >= key_m; a funnel shift moves each sign bit in.
__device__ __forceinline__ uint32_t cmp6(uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
  uint32_t c = 0;
  c = __funnelshift_l(k1 - k0 - 1u, c, 1);
  c = __funnelshift_l(k2 - k0 - 1u, c, 1);
  c = __funnelshift_l(k3 - k0 - 1u, c, 1);
  c = __funnelshift_l(k2 - k1 - 1u, c, 1);
  c = __funnelshift_l(k3 - k1 - 1u, c, 1);
  c = __funnelshift_l(k3 - k2 - 1u, c, 1);
  return c;
}

// {hi, lo} -> packed bf16x2, round to nearest even (NaN comes out as 0x7fff: see slots()).
__device__ __forceinline__ uint32_t cvt_bf16x2(float hi, float lo) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// The two bf16 slots of a block from its table entry.  Fast path: two packed conversions and
// one byte permute; a block that holds a NaN takes the exact integer conversion instead so that
// the NaN payload rule (quiet bit set, sign and top payload bits kept) holds bit for bit.
// CHECK_NAN = false: the caller has already established that none of the four is a NaN.
template <bool BOTH_KEPT, bool CHECK_NAN = true>
__device__ __forceinline__ uint32_t slots(uint32_t e, float w0, float w1, float w2, float w3,
                                          uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
  if (CHECK_NAN && max(max(k0, k1), max(k2, k3)) > 0x7F800000u) {
    const uint32_t idx0 = (e >> 4) & 3u, idx1 = (e >> 6) & 3u;
    const float s0 = idx0 == 0 ? w0 : idx0 == 1 ? w1 : w2;      // idx0 is never 3
    const float s1 = idx1 == 1 ? w1 : idx1 == 2 ? w2 : w3;      // idx1 is never 0
    const uint32_t a = (e & 0x100u) ? to_bf16(s0) : 0u;
    const uint32_t b = (e & 0x200u) ? to_bf16(s1) : 0u;
    return a | (b << 16);
  }
  uint32_t v = __byte_perm(cvt_bf16x2(w1, w0), cvt_bf16x2(w3, w2), e >> 16);
  if (!BOTH_KEPT) v &= (((e >> 8) & 1u) * 0xFFFFu) | (((e >> 9) & 1u) * 0xFFFF0000u);
  return v;
}

// The two bf16 slots of a block from an entry of lut_entry_signs: two packed conversions and three byte permutes
// (select the slots; expand the two "kept" bits into a mask).  A block that holds a NaN takes the exact integer
// conversion (see slots()).
__device__ __forceinline__ uint32_t slots_signs(uint32_t e, float w0, float w1, float w2, float w3,
                                                uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
  uint32_t keep;                                           // bytes 0-1: sign of byte 3, bytes 2-3: sign of byte 2
  asm("prmt.b32 %0, %1, %1, 0xAABB;" : "=r"(keep) : "r"(e));
  if (max(max(k0, k1), max(k2, k3)) > 0x7F800000u) {
    const uint32_t idx0 = (e >> 24) & 3u, idx1 = (e >> 26) & 3u;
    const float s0 = idx0 == 0 ? w0 : idx0 == 1 ? w1 : w2;      // idx0 is never 3
    const float s1 = idx1 == 1 ? w1 : idx1 == 2 ? w2 : w3;      // idx1 is never 0
    return (to_bf16(s0) | (to_bf16(s1) << 16)) & keep;
  }
  return __byte_perm(cvt_bf16x2(w1, w0), cvt_bf16x2(w3, w2), e) & keep;
}

// The optimizer update fused into a forward-mask pass (fp32, every operation rounded once, in this order:
//   g = dW + weight_decay * W ;  mom = momentum * mom + g ;  W = W - lr * mom).
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

// One canonical code word (row r of the packed operand, 32-column word w) scattered into the
// tensor-memory image of the metadata (one 2048-byte block per 128 rows x 128 k: 128 lanes x 4
// columns of u32, lane = m0 + 8*h + 16*m2 holding rows m0 + 16*m2 / + 8 of k-half h): its low 16 bits (k-half 0) and high 16 bits
// (k-half 1) land in two different lanes, each as one half of a 32-bit word whose other half
// comes from the row 8 above or below.  Used when the operand has no padding (rows and K both
// multiples of 128), so that the separate re-ordering pass is not needed.
__device__ __forceinline__ void scatter_hw(uint16_t* __restrict__ hw16, int tiles_k, int r, int w, uint32_t word) {
  const int rr = r & 127;
  const size_t tile = (size_t)(r >> 7) * tiles_k + (w >> 2);
  const size_t idx = (tile * 512 + (size_t)((rr & 7) + 16 * (rr >> 4)) * 4 + (w & 3)) * 2 + ((rr >> 3) & 1);
  hw16[idx] = (uint16_t)(word & 0xFFFFu);
  hw16[idx + 64] = (uint16_t)(word >> 16);               // lane + 8: 8 lanes x 4 words x 2 halves
}

// Padding of the tensor-memory image (operands whose rows or k extent are not multiples of 128): every 32-bit entry
// that belongs wholly to rows >= rows or code words >= kwords gets the harmless code 0x4 (slots (0, 1); the values
// there are zero).  rows % 16 == 0, so an entry (two rows eight apart) is never half real.  Called by all threads of
// a grid (tid of nthreads); the real entries are written by the mask kernels themselves.
__device__ __forceinline__ void pad_hw_image(uint32_t* __restrict__ hw32, int rows, int kwords, long long tid, long long nthreads) {
  const int tiles_k = (kwords + 3) >> 2;
  const long long n = (long long)((rows + 127) >> 7) * tiles_k * 512;
  for (long long e = tid; e < n; e += nthreads) {
    const long long tile = e >> 9;
    const int L = (int)(e & 511) >> 2, kc = (int)(e & 3);
    const int mt = (int)(tile / tiles_k), kt = (int)(tile - (long long)mt * tiles_k);
    const int r_lo = mt * 128 + (L & 7) + 16 * (L >> 4);
    if (r_lo >= rows || kt * 4 + kc >= kwords) hw32[e] = 0x44444444u;
  }
}

}  // namespace
}  // namespace bimask
