// N:M patterns beyond 2:4 and 1:4 (the paper also trains 4:8, 2:8, 1:8 and 1:16): forward mask,
// eligible-block count and backward mask for block lengths M = 8 and 16.  Selection is the same
// rank rule as for M = 4 (an element is kept when fewer than N candidates of its block beat it;
// ties go to the lower index), evaluated in registers (see keep_block).
// When N <= 2 every aligned group of four holds at most two survivors, so the result is packed
// into the same 2:4 tensor-core operand as before (the index code of a group depends on its keep
// mask alone); patterns with N > 2 (4:8) produce mask bits only.
#include "common.cuh"
#include "mask_common.cuh"

namespace bimask {

namespace {

// keep mask of one block of M keys: bit m set iff candidate m is beaten by fewer than N candidates
// (q beats m when key_q > key_m, or key_q == key_m with q < m).
//   N <= 2: N rounds of "largest remaining candidate, lowest index on ties" -- about 5 M operations
//           per round instead of all M (M - 1) / 2 pairwise comparisons;
//   N  > 2: threshold = the N-th largest key, found by a sorting network (below).
template <int M>
__device__ __forceinline__ uint32_t keep_block(const uint32_t (&key)[M], uint32_t valid, int N) {
  uint32_t kb = 0;
  if (N <= 2) {
    uint32_t k[M];                                        // 0 = not a candidate (keys are < 2^31, so +1 fits)
#pragma unroll
    for (int m = 0; m < M; ++m) k[m] = ((valid >> m) & 1u) ? key[m] + 1u : 0u;
#pragma unroll
    for (int round = 0; round < 2; ++round) {
      if (round < N) {
        uint32_t mx = k[0];
#pragma unroll
        for (int m = 1; m < M; ++m) mx = max(mx, k[m]);
        uint32_t eq = 0;
#pragma unroll
        for (int m = 0; m < M; ++m) eq |= (k[m] == mx ? 1u : 0u) << m;
        const uint32_t pick = mx ? (eq & (0u - eq)) : 0u;  // lowest index among the largest; none if no candidate is left
        kb |= pick;
        if (round == 0) {
#pragma unroll
          for (int m = 0; m < M; ++m) k[m] = ((pick >> m) & 1u) ? 0u : k[m];
        }
      }
    }
    return kb;
  }
  // N > 2: the N-th largest candidate key t from a sorting network on the keys alone (bitonic, min / max pairs with
  // compile-time indices: 24 pairs for M = 8, 80 for M = 16, against M (M - 1) / 2 pairwise comparisons with two
  // conditional increments each); kept are the candidates above t and, of those equal to t, the lowest indices up
  // to N in all -- which is the rank rule: q beats m when key_q > key_m, or key_q == key_m with q < m.
  uint32_t k[M], srt[M];                                  // 0 = not a candidate (keys are < 2^31, so +1 fits)
#pragma unroll
  for (int m = 0; m < M; ++m) k[m] = srt[m] = ((valid >> m) & 1u) ? key[m] + 1u : 0u;
#pragma unroll
  for (int span = 2; span <= M; span <<= 1)
#pragma unroll
    for (int j = span >> 1; j > 0; j >>= 1)
#pragma unroll
      for (int i = 0; i < M; ++i) {
        const int l = i ^ j;
        if (l > i) {
          const uint32_t lo = min(srt[i], srt[l]), hi = max(srt[i], srt[l]);
          const bool descending = (i & span) == 0;        // the whole array ends up in descending order
          srt[i] = descending ? hi : lo;
          srt[l] = descending ? lo : hi;
        }
      }
  uint32_t t = srt[0];
#pragma unroll
  for (int m = 1; m < M; ++m) t = (m == N - 1) ? srt[m] : t;
  uint32_t ge = 0;
#pragma unroll
  for (int m = 0; m < M; ++m) ge |= (k[m] >= t ? 1u : 0u) << m;
  // the usual cases: no tie at the threshold (exactly N at or above it), or fewer than N candidates (t == 0: all of
  // them are kept).  Taken only when every lane of the warp is in one of them (every caller runs whole warps).
  if (__all_sync(0xFFFFFFFFu, t == 0u || __popc(ge) == N)) return t == 0u ? valid : ge;
  uint32_t gt = 0, eq = 0;
#pragma unroll
  for (int m = 0; m < M; ++m) {
    gt |= (k[m] > t ? 1u : 0u) << m;
    eq |= (k[m] == t ? 1u : 0u) << m;
  }
  eq &= valid;                                            // t == 0: fewer than N candidates, all of them are above it
  kb = gt;
  int need = N - __popc(gt);
#pragma unroll
  for (int i = 0; i < M; ++i) {
    if (i < N && need > 0) {
      const uint32_t b = eq & (0u - eq);
      kb |= b;
      eq ^= b;
      --need;
    }
  }
  return kb;
}

// ---------------------------------------------------------------------------------------
// Forward mask (+ pack when PACK).  One lane per block of M consecutive weights; the 32 / M lanes
// that share a 32-column word OR their pieces together.
// ---------------------------------------------------------------------------------------
// MODE 0: mask bits only; 1: 2:4 operand (values + index codes); 2: dense masked bf16 operand
// (kept weights rounded to bf16, +0 elsewhere) for patterns the 2:4 format cannot hold.
// (blocks of sixteen weights per lane would take 104-115 registers: two CTAs per SM, a quarter of the warps an SM can
// hold, for kernels that live on hiding load latency.  Measured at 1:16 on 16384 x 4096: forward mask 168 us
// unbounded, 131 us at three CTAs per SM, 123 us at four (64 registers, a few dozen bytes of spills); the backward
// mask is best at three)
// UPDATE: the optimizer update of Alg. 1 applied to the block as it is loaded (W, dW and the momentum buffer are read,
// W and the momentum buffer written back), so that the next iteration's mask costs no second pass over W.
template <int M, int MODE, bool UPDATE = false>
__global__ void __launch_bounds__(256, 4)
fwd_mask_generic_kernel(const float4* __restrict__ W4, long long nblocks, int N,
                        uint32_t* __restrict__ maskbits, uint32_t* __restrict__ vals32,
                        uint32_t* __restrict__ meta, uint16_t* __restrict__ hw16, int jwords, SgdParams sgd) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int LPW = 32 / M;                               // lanes per 32-column word
  constexpr int G = M / 4;                                  // groups of four per block
  __shared__ uint32_t pad16[16];                            // container entry of a group from its keep mask
  if (threadIdx.x < 16) pad16[threadIdx.x] = lut_entry(0u, threadIdx.x, 4);
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const uint32_t gmask = ((LPW == 4 ? 0xFu : 0x3u)) << (lane & ~(LPW - 1));
  const int sh = M * (lane & (LPW - 1));
  const long long stride = (long long)gridDim.x * blockDim.x;
  const long long nround = (nblocks + 31) & ~31ll;          // whole warps stay in the loop together
  // the next trip's block is loaded before this trip's is worked on (one block of loads always in flight)
  float4 nxt[UPDATE ? 1 : G];
  if (!UPDATE) {
    const long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x;
#pragma unroll
    for (int g = 0; g < G; ++g) nxt[g] = b < nblocks ? __ldg(W4 + b * G + g) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (long long b = (long long)blockIdx.x * blockDim.x + threadIdx.x; b < nround; b += stride) {
    const bool live = b < nblocks;
    float w[M];
    if (UPDATE) {
      // three streams in, two out; no look-ahead (it would triple the registers held across the trip)
      float4 wv[G], dv[G], mv[G];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        wv[g] = live ? sgd.W4[b * G + g] : make_float4(0.f, 0.f, 0.f, 0.f);
        dv[g] = live ? __ldg(sgd.dW4 + b * G + g) : make_float4(0.f, 0.f, 0.f, 0.f);
        mv[g] = (live && sgd.mom4) ? sgd.mom4[b * G + g] : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        wv[g].x = sgd_one(wv[g].x, dv[g].x, mv[g].x, sgd);
        wv[g].y = sgd_one(wv[g].y, dv[g].y, mv[g].y, sgd);
        wv[g].z = sgd_one(wv[g].z, dv[g].z, mv[g].z, sgd);
        wv[g].w = sgd_one(wv[g].w, dv[g].w, mv[g].w, sgd);
        if (live) {
          sgd.W4[b * G + g] = wv[g];
          if (sgd.mom4) sgd.mom4[b * G + g] = mv[g];
        }
        w[4 * g] = wv[g].x; w[4 * g + 1] = wv[g].y; w[4 * g + 2] = wv[g].z; w[4 * g + 3] = wv[g].w;
      }
    } else {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float4 v = nxt[g];
        w[4 * g] = v.x; w[4 * g + 1] = v.y; w[4 * g + 2] = v.z; w[4 * g + 3] = v.w;
      }
      const long long bn = b + stride;
#pragma unroll
      for (int g = 0; g < G; ++g) nxt[g] = bn < nblocks ? __ldg(W4 + bn * G + g) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    uint32_t key[M];
#pragma unroll
    for (int m = 0; m < M; ++m) key[m] = mag_key(w[m]);
    const uint32_t kb = keep_block<M>(key, (M == 16 ? 0xFFFFu : 0xFFu), N);
    uint32_t codes = 0;
    if (MODE == 1) {
      uint32_t pv[G];                                     // the block's G packed pairs: one 8- or 16-byte store
      uint32_t mxk = key[0];
#pragma unroll
      for (int m = 1; m < M; ++m) mxk = max(mxk, key[m]);
      // one NaN test per warp trip instead of a branch per group of four (a NaN takes the exact integer conversion)
      if (__any_sync(0xFFFFFFFFu, mxk > 0x7F800000u)) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const uint32_t e = pad16[(kb >> (4 * g)) & 15u];
          pv[g] = slots<false, true>(e, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3], key[4 * g], key[4 * g + 1],
                                     key[4 * g + 2], key[4 * g + 3]);
          codes |= ((e >> 4) & 15u) << (4 * g);
        }
      } else {
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const uint32_t e = pad16[(kb >> (4 * g)) & 15u];
          pv[g] = slots<false, false>(e, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3], 0u, 0u, 0u, 0u);
          codes |= ((e >> 4) & 15u) << (4 * g);
        }
      }
      if (live) {
        if (G == 2) reinterpret_cast<uint2*>(vals32)[b] = make_uint2(pv[0], pv[1]);
        else reinterpret_cast<uint4*>(vals32)[b] = make_uint4(pv[0], pv[1], pv[G > 2 ? 2 : 0], pv[G > 3 ? 3 : 0]);
      }
    }
    if (MODE == 2 && live) {
      uint4* dst = reinterpret_cast<uint4*>(vals32) + b * (M / 8);
      uint32_t mx = key[0];
#pragma unroll
      for (int m = 1; m < M; ++m) mx = max(mx, key[m]);
      const bool has_nan = mx > 0x7F800000u;              // the packed conversion would canonicalise a NaN's payload
#pragma unroll
      for (int h = 0; h < M / 8; ++h) {
        uint32_t d[4];
        if (has_nan) {
#pragma unroll
          for (int j = 0; j < 4; ++j) d[j] = to_bf16(w[8 * h + 2 * j]) | (to_bf16(w[8 * h + 2 * j + 1]) << 16);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) d[j] = cvt_bf16x2(w[8 * h + 2 * j + 1], w[8 * h + 2 * j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t f = (kb >> (8 * h + 2 * j)) & 3u;  // kept bits of the pair -> 16-bit masks
          d[j] &= (f & 1u) * 0xFFFFu + (f >> 1) * 0xFFFF0000u;
        }
        dst[h] = make_uint4(d[0], d[1], d[2], d[3]);
      }
    }
    const uint32_t wb = __reduce_or_sync(gmask, kb << sh);
    const uint32_t wm = __reduce_or_sync(gmask, codes << sh);
    if (live && (lane & (LPW - 1)) == 0) {
      const long long word = b / LPW;
      maskbits[word] = wb;
      if (MODE == 1) {
        meta[word] = wm;
        if (hw16) {                                         // unpadded operand: write the tensor-memory image here
          const int r = (int)(word / jwords);
          scatter_hw(hw16, jwords >> 2, r, (int)(word - (long long)r * jwords), wm);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Eligible-block count for blocks of M permuted rows: a column is eligible when at most N of the
// M rows have its bit set.  Bit-sliced saturating counter: level[j] = "at least j rows so far".
// ---------------------------------------------------------------------------------------
template <int N>
struct SatCount {
  uint32_t lv[N + 1];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int j = 0; j <= N; ++j) lv[j] = 0u;
  }
  __device__ __forceinline__ void add(uint32_t x) {
#pragma unroll
    for (int j = N; j >= 1; --j) lv[j] |= lv[j - 1] & x;
    lv[0] |= x;
  }
  __device__ __forceinline__ uint32_t eligible() const { return ~lv[N]; }   // fewer than N + 1 rows set
};

template <int N, int M>
__global__ void __launch_bounds__(256)
score_generic_kernel(const uint32_t* __restrict__ bits, const int32_t* __restrict__ cands, int I, int jwords,
                     int blocks_per_cta, unsigned long long* __restrict__ counts) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.y;
  const int nblk = I / M;
  const int b0 = blockIdx.x * blocks_per_cta;
  const int b1 = min(nblk, b0 + blocks_per_cta);
  const int32_t* cand = cands + (long long)c * I;
  const unsigned last_row = (unsigned)(I - 1);
  uint32_t cnt = 0;
  for (int b = b0 + warp; b < b1; b += 8) {
    int rows[M];
#pragma unroll
    for (int g = 0; g < M / 4; ++g) {
      const int4 r = __ldg(reinterpret_cast<const int4*>(cand + (long long)b * M) + g);
      rows[4 * g] = checked_row(r.x, (int)last_row + 1, SITE_GENERIC_CAND); rows[4 * g + 1] = checked_row(r.y, (int)last_row + 1, SITE_GENERIC_CAND);
      rows[4 * g + 2] = checked_row(r.z, (int)last_row + 1, SITE_GENERIC_CAND); rows[4 * g + 3] = checked_row(r.w, (int)last_row + 1, SITE_GENERIC_CAND);
    }
    if ((jwords & 3) == 0) {
      // 128-bit loads: four words of every row at once (a quarter of the load instructions)
      const int jq = jwords >> 2;
      for (int q = lane; q < jq; q += 32) {
        SatCount<N> s0, s1, s2, s3;
        s0.clear(); s1.clear(); s2.clear(); s3.clear();
#pragma unroll
        for (int m = 0; m < M; ++m) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(bits + (long long)rows[m] * jwords) + q);
          s0.add(v.x); s1.add(v.y); s2.add(v.z); s3.add(v.w);
        }
        cnt += __popc(s0.eligible()) + __popc(s1.eligible()) + __popc(s2.eligible()) + __popc(s3.eligible());
      }
    } else {
      for (int q = lane; q < jwords; q += 32) {
        SatCount<N> s;
        s.clear();
#pragma unroll
        for (int m = 0; m < M; ++m) s.add(__ldg(bits + (long long)rows[m] * jwords + q));
        cnt += __popc(s.eligible());
      }
    }
  }
  cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
  __shared__ uint32_t part[8];
  if (lane == 0) part[warp] = cnt;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long s = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += part[w];
    atomicAdd(counts + c, s);
  }
}

// ---------------------------------------------------------------------------------------
// Greedy refinement of a permutation by pairwise swaps (hill climbing on the eligible-block
// count; not part of the paper's Algorithm 1, which stops at the best random candidate).
// A round pairs the positions of the permutation at random: pair i = (order[2i], order[2i+1]).
// gain kernel: one warp per pair; lanes stride over the 32-column words; for each word the M
// mask words of both row blocks are loaded once and the eligible columns counted before and after
// exchanging the two rows.  A pair with positive gain bids for both of its blocks with
// (gain << 32 | ~pair index) through a 64-bit atomic maximum.
// apply kernel: a pair that won BOTH of its blocks exchanges its two entries of perm; winners never
// share a block, so their gains add up and a round never lowers the count.
// ---------------------------------------------------------------------------------------
template <int N, int M>
__global__ void __launch_bounds__(256)
refine_gain_kernel(const uint32_t* __restrict__ bits, const int32_t* __restrict__ perm, const int32_t* __restrict__ order,
                   int I, int jwords, int32_t* __restrict__ gains, unsigned long long* __restrict__ block_best) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int pair = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (pair >= (I >> 1)) return;
  const int a = __ldg(order + 2 * pair), b = __ldg(order + 2 * pair + 1);
  const int ka = a / M, kb = b / M;
  if (ka == kb) {
    if (lane == 0) gains[pair] = 0;
    return;
  }
  const unsigned last_row = (unsigned)(I - 1);
  int ra[M], rb[M];
#pragma unroll
  for (int m = 0; m < M; ++m) {
    ra[m] = checked_row(__ldg(perm + ka * M + m), (int)last_row + 1, SITE_GENERIC_PERM);
    rb[m] = checked_row(__ldg(perm + kb * M + m), (int)last_row + 1, SITE_GENERIC_PERM);
  }
  const int ma = a - ka * M, mb = b - kb * M;
  int gain = 0;
  for (int q = lane; q < jwords; q += 32) {
    uint32_t wa[M], wb[M];
#pragma unroll
    for (int m = 0; m < M; ++m) {
      wa[m] = __ldg(bits + (long long)ra[m] * jwords + q);
      wb[m] = __ldg(bits + (long long)rb[m] * jwords + q);
    }
    uint32_t xa = 0, xb = 0;                                 // the two rows that change places
#pragma unroll
    for (int m = 0; m < M; ++m) {
      xa = m == ma ? wa[m] : xa;
      xb = m == mb ? wb[m] : xb;
    }
    SatCount<N> s0, s1, s2, s3;
    s0.clear(); s1.clear(); s2.clear(); s3.clear();
#pragma unroll
    for (int m = 0; m < M; ++m) {
      s0.add(wa[m]);
      s1.add(wb[m]);
      s2.add(m == ma ? xb : wa[m]);
      s3.add(m == mb ? xa : wb[m]);
    }
    gain += __popc(s2.eligible()) + __popc(s3.eligible()) - __popc(s0.eligible()) - __popc(s1.eligible());
  }
  gain = __reduce_add_sync(0xFFFFFFFFu, gain);
  if (lane == 0) {
    gains[pair] = gain;
    if (gain > 0) {
      const unsigned long long key = ((unsigned long long)(unsigned)gain << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)pair);
      atomicMax(block_best + ka, key);
      atomicMax(block_best + kb, key);
    }
  }
}

template <int M>
__global__ void refine_apply_kernel(const int32_t* __restrict__ order, const int32_t* __restrict__ gains,
                                    const unsigned long long* __restrict__ block_best, int I, int32_t* __restrict__ perm) {
  pdl_launch_dependents();
  pdl_wait();
  const int pair = blockIdx.x * blockDim.x + threadIdx.x;
  if (pair >= (I >> 1)) return;
  const int gain = gains[pair];
  if (gain <= 0) return;
  const int a = __ldg(order + 2 * pair), b = __ldg(order + 2 * pair + 1);
  const unsigned long long key = ((unsigned long long)(unsigned)gain << 32) | (unsigned long long)(0xFFFFFFFFu - (unsigned)pair);
  if (block_best[a / M] == key && block_best[b / M] == key) {
    const int32_t pa = perm[a], pb = perm[b];
    perm[a] = pb;
    perm[b] = pa;
  }
}

__global__ void fill_counts_kernel(long long* counts, int P, long long v) {
  pdl_launch_dependents();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < P) counts[i] = v;
}

// ---------------------------------------------------------------------------------------
// Backward mask (+ transposed pack when PACK).  A warp owns 32 permuted rows x 32 columns (lane =
// column): 32 / M blocks of M rows, which is exactly one metadata word and one 32-byte sector of
// packed values per column.  Rows are gathered with one coalesced 128-byte load each.
// ---------------------------------------------------------------------------------------
// Criteria of the paper's ablation on how the backward mask picks its N survivors (Sec. 4.4):
// 0 weight magnitude (Eq. 11), 1 magnitude of another matrix S (the weight gradient), 2 N draws
// without replacement proportional to |w|, 3 random.  Whatever the criterion only entries whose
// forward bit is set compete, and a block with at most N competitors keeps them all.
__device__ __forceinline__ uint64_t mix64_dev(uint64_t z) {
  z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27; z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

// Draw number d takes the first remaining competitor whose running sum of |w| exceeds u * total
// (u: 24 random bits, a function of seed, d and the block index); the lowest remaining one when
// none does.  float32, each operation rounded once, sums in row order: reproducible bit for bit.
template <int M>
__device__ __forceinline__ uint32_t multinomial_block(const float (&w)[M], uint32_t valid, int N, uint64_t seed,
                                                      uint64_t block_index) {
  if (__popc(valid) <= N) return valid;
  uint32_t rem = valid, keep = 0;
  for (int d = 0; d < N; ++d) {
    const uint64_t h = mix64_dev(mix64_dev(seed + 0x9E3779B97F4A7C15ull * (uint64_t)(d + 1)) ^ block_index);
    const float u = __fmul_rn(__uint2float_rn((uint32_t)(h >> 40)), 5.9604644775390625e-8f);   // * 2^-24, exact
    float total = 0.f;
#pragma unroll
    for (int m = 0; m < M; ++m)
      if ((rem >> m) & 1u) total = __fadd_rn(total, fabsf(w[m]));
    const float x = __fmul_rn(u, total);
    float cum = 0.f;
    int chosen = -1;
#pragma unroll
    for (int m = 0; m < M; ++m)
      if ((rem >> m) & 1u) {
        cum = __fadd_rn(cum, fabsf(w[m]));
        if (chosen < 0 && cum > x) chosen = m;
      }
    if (chosen < 0) chosen = __ffs(rem) - 1;
    keep |= 1u << chosen;
    rem &= ~(1u << chosen);
  }
  return keep;
}

// Passes (groups of 32 permuted rows) a warp handles per trip: as many as make a column's share of the operand a
// whole 128-byte line (32 B per pass in the 2:4 container, 64 B per pass in the dense operand).
template <int MODE>
struct BwdGenericTrip { static constexpr int PASSES = MODE == 2 ? 2 : 4; };

template <int M, int MODE, int CRIT>
__global__ void __launch_bounds__(256, M == 16 ? 3 : 4)
bwd_mask_generic_kernel(const float* __restrict__ W, const uint32_t* __restrict__ maskbits_f,
                        const int32_t* __restrict__ perm, int I, int J, int N,
                        uint32_t* __restrict__ maskbits_b, uint32_t* __restrict__ vals_b,
                        uint32_t* __restrict__ meta_b, const float* __restrict__ S, uint64_t seed,
                        uint16_t* __restrict__ hw16) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int NB = 32 / M;                                // blocks per 32-row pass
  constexpr int G = M / 4;
  constexpr int PP = BwdGenericTrip<MODE>::PASSES;
  __shared__ uint32_t pad16[16];
  // operand rows are columns of W: a lane's results of one pass are 32 or 64 bytes of ITS row, so stored from
  // registers every instruction of a warp would touch 32 lines.  They are staged per warp as [32 columns][eight
  // 16-byte units] (unit index XOR column mod 8: conflict-free 16-byte stores and loads) over PP passes and written
  // out as whole 128-byte lines, four columns per instruction.
  __shared__ uint4 stage_all[MODE == 0 ? 1 : 8 * 256];
  __shared__ uint32_t code_all[MODE == 1 ? 8 * 32 * 4 : 1];
  if (threadIdx.x < 16) pad16[threadIdx.x] = lut_entry(0u, threadIdx.x, 4);
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int jwords = J >> 5;
  const int cw = blockIdx.y * 8 + warp;                     // column word of this warp
  if (cw >= jwords) return;
  const int col = 32 * cw + lane;
  const int npass = I >> 5, pass0 = blockIdx.x * PP;
  const int done = npass - pass0 < PP ? npass - pass0 : PP; // passes of this trip
  uint4* stage = stage_all + (MODE == 0 ? 0 : warp * 256);
  uint32_t* codes = code_all + (MODE == 1 ? warp * 128 : 0);
#pragma unroll 1
  for (int pp = 0; pp < done; ++pp) {
    const int pass = pass0 + pp;                            // 32 permuted rows
    const int my_src = checked_row(__ldg(perm + 32 * pass + lane), I, SITE_GENERIC_PERM);   // lane r: source of permuted row r
    // lane r loads the forward-mask word of permuted row r; one 32 x 32 bit transpose gives every lane (= column) the
    // candidate bits of its column in the 32 rows, and the kept bits go back to row words the same way
    const uint32_t cand = transpose32(__ldg(maskbits_f + (size_t)my_src * jwords + cw), lane);
    uint32_t colkeep = 0;
    uint32_t vacc[8];
    uint32_t dacc[MODE == 2 ? 16 : 1];                      // dense: this column's 32 permuted rows as bf16 pairs
    uint32_t cacc = 0;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      float w[M];
      uint32_t key[M];                                      // magnitude of the weight (values, NaN handling)
      uint32_t skey[(CRIT == 1 || CRIT == 3) ? M : 1];      // what the criterion ranks by
      const uint32_t valid = (cand >> (nb * M)) & ((1u << M) - 1u);
#pragma unroll
      for (int m = 0; m < M; ++m) {
        const int src = __shfl_sync(0xFFFFFFFFu, my_src, nb * M + m);
        w[m] = __ldg(W + (size_t)src * J + col);
        key[m] = mag_key(w[m]);
        if constexpr (CRIT == 1) skey[m] = mag_key(__ldg(S + (size_t)src * J + col));
        if constexpr (CRIT == 3) skey[m] = (uint32_t)(mix64_dev(seed + (uint64_t)src * (uint64_t)J + (uint64_t)col) >> 33);
      }
      uint32_t kb;
      if constexpr (CRIT == 0) kb = keep_block<M>(key, valid, N);
      else if constexpr (CRIT == 2) kb = multinomial_block<M>(w, valid, N, seed, (uint64_t)(pass * NB + nb) * (uint64_t)J + (uint64_t)col);
      else kb = keep_block<M>(skey, valid, N);
      colkeep |= kb << (nb * M);
      if (MODE == 2) {
#pragma unroll
        for (int m = 0; m < M; m += 2) {
          const uint32_t lo = ((kb >> m) & 1u) ? to_bf16(w[m]) : 0u;
          const uint32_t hi = ((kb >> (m + 1)) & 1u) ? to_bf16(w[m + 1]) : 0u;
          dacc[(nb * M + m) / 2] = lo | (hi << 16);
        }
      }
      if (MODE == 1) {
        uint32_t mxk = key[0];
#pragma unroll
        for (int m = 1; m < M; ++m) mxk = max(mxk, key[m]);
        const bool nan_here = __any_sync(0xFFFFFFFFu, mxk > 0x7F800000u);   // one test per warp and block row
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const uint32_t e = pad16[(kb >> (4 * g)) & 15u];
          vacc[nb * G + g] = nan_here ? slots<false, true>(e, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3], key[4 * g],
                                                           key[4 * g + 1], key[4 * g + 2], key[4 * g + 3])
                                      : slots<false, false>(e, w[4 * g], w[4 * g + 1], w[4 * g + 2], w[4 * g + 3], 0u, 0u, 0u, 0u);
          cacc |= ((e >> 4) & 15u) << (4 * (nb * G + g));
        }
      }
    }
    maskbits_b[(size_t)(32 * pass + lane) * jwords + cw] = transpose32(colkeep, lane);
    if (MODE == 1) {
      stage[lane * 8 + ((2 * pp) ^ (lane & 7))] = make_uint4(vacc[0], vacc[1], vacc[2], vacc[3]);
      stage[lane * 8 + ((2 * pp + 1) ^ (lane & 7))] = make_uint4(vacc[4], vacc[5], vacc[6], vacc[7]);
      codes[lane * 4 + pp] = cacc;
      if (hw16) scatter_hw(hw16, I >> 7, col, pass, cacc);
    }
    if (MODE == 2) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        stage[lane * 8 + ((4 * pp + q) ^ (lane & 7))] = make_uint4(dacc[4 * q], dacc[4 * q + 1], dacc[4 * q + 2], dacc[4 * q + 3]);
    }
  }
  if (MODE != 0) {
    __syncwarp();
    // row `c` of the J x I operand, the trip's 16-byte units u = 0 .. 8 done / PP - 1: four columns per instruction
    const int units = done * (8 / PP);
    const size_t row_words = MODE == 1 ? (size_t)(I >> 2) : (size_t)(I >> 1);
    const int u = lane & 7;
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int c = 4 * it + (lane >> 3);
      if (u < units)
        reinterpret_cast<uint4*>(vals_b + (size_t)(32 * cw + c) * row_words + (size_t)pass0 * (MODE == 1 ? 8 : 16))[u] =
            stage[c * 8 + (u ^ (c & 7))];
    }
    if (MODE == 1) {                                        // the trip's index-code words of this lane's column
      uint32_t* dst = meta_b + (size_t)col * (I >> 5) + pass0;
      if (done == 4 && (I & 127) == 0) {
        *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(codes + lane * 4);
      } else {
        for (int pp = 0; pp < done; ++pp) dst[pp] = codes[lane * 4 + pp];
      }
    }
  }
}

}  // namespace

BIMASK_DEFINE_DEBUG_COLLECT(debug_collect_generic)

// mode: 0 mask bits only, 1 the 2:4 operand, 2 the dense masked operand (written to `vals`)
template <int M, bool UPDATE>
static int launch_fwd_generic_m(int mode, unsigned ctas, cudaStream_t s, const float4* W4, long long nblocks, int N, uint32_t* maskbits,
                                uint32_t* v32, uint32_t* meta, uint16_t* hw16, int jw, const SgdParams& sgd) {
  if (mode == 1) BIMASK_CUDA_OK(launch_pdl(fwd_mask_generic_kernel<M, 1, UPDATE>, ctas, 256, 0, s, W4, nblocks, N, maskbits, v32, meta, hw16, jw, sgd));
  else if (mode == 2) BIMASK_CUDA_OK(launch_pdl(fwd_mask_generic_kernel<M, 2, UPDATE>, ctas, 256, 0, s, W4, nblocks, N, maskbits, v32, meta, hw16, jw, sgd));
  else BIMASK_CUDA_OK(launch_pdl(fwd_mask_generic_kernel<M, 0, UPDATE>, ctas, 256, 0, s, W4, nblocks, N, maskbits, v32, meta, hw16, jw, sgd));
  return BIMASK_OK;
}

// dW != nullptr: the optimizer update (lr, momentum, weight_decay; mom_or_null) is applied to W on the way.
int launch_fwd_mask_generic(const float* W, int I, int J, int N, int M, uint32_t* maskbits, uint16_t* vals_or_null,
                            uint32_t* meta_or_null, int mode, void* hw_meta_or_null, cudaStream_t s, const float* dW,
                            float* mom_or_null, float lr, float momentum, float weight_decay) {
  uint16_t* hw16 = reinterpret_cast<uint16_t*>(hw_meta_or_null);
  const int jw = J / 32;
  const long long nblocks = (long long)I * J / M;
  long long ctas = (nblocks + 255) / 256;
  if (ctas > 148 * 16) ctas = 148 * 16;
  const float4* W4 = reinterpret_cast<const float4*>(W);
  uint32_t* v32 = reinterpret_cast<uint32_t*>(vals_or_null);
  const SgdParams sgd{reinterpret_cast<float4*>(const_cast<float*>(W)), reinterpret_cast<const float4*>(dW),
                      reinterpret_cast<float4*>(mom_or_null), lr, momentum, weight_decay};
  int rc;
  if (dW) rc = M == 8 ? launch_fwd_generic_m<8, true>(mode, (unsigned)ctas, s, W4, nblocks, N, maskbits, v32, meta_or_null, hw16, jw, sgd)
                      : launch_fwd_generic_m<16, true>(mode, (unsigned)ctas, s, W4, nblocks, N, maskbits, v32, meta_or_null, hw16, jw, sgd);
  else rc = M == 8 ? launch_fwd_generic_m<8, false>(mode, (unsigned)ctas, s, W4, nblocks, N, maskbits, v32, meta_or_null, hw16, jw, sgd)
                   : launch_fwd_generic_m<16, false>(mode, (unsigned)ctas, s, W4, nblocks, N, maskbits, v32, meta_or_null, hw16, jw, sgd);
  if (rc != BIMASK_OK) return rc;
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

template <int M>
static int launch_score_m(const uint32_t* bits, const int32_t* cands, int I, int J, int N, int P, int64_t* counts,
                          cudaStream_t s) {
  const int nblk = I / M;
  const int per_cta = 64;
  dim3 grid((nblk + per_cta - 1) / per_cta, P);
  unsigned long long* cnt = reinterpret_cast<unsigned long long*>(counts);
  switch (N) {
    case 1: BIMASK_CUDA_OK(launch_pdl(score_generic_kernel<1, M>, grid, 256, 0, s, bits, cands, I, J / 32, per_cta, cnt)); break;
    case 2: BIMASK_CUDA_OK(launch_pdl(score_generic_kernel<2, M>, grid, 256, 0, s, bits, cands, I, J / 32, per_cta, cnt)); break;
    case 3: BIMASK_CUDA_OK(launch_pdl(score_generic_kernel<3, M>, grid, 256, 0, s, bits, cands, I, J / 32, per_cta, cnt)); break;
    default: BIMASK_CUDA_OK(launch_pdl(score_generic_kernel<4, M>, grid, 256, 0, s, bits, cands, I, J / 32, per_cta, cnt)); break;
  }
  return BIMASK_OK;
}

int launch_score_generic(const uint32_t* bits, const int32_t* cands, int I, int J, int N, int M, int P,
                         int64_t* counts, cudaStream_t s) {
  if (N >= M) {                                             // every block is eligible
    BIMASK_CUDA_OK(launch_pdl(fill_counts_kernel, (P + 255) / 256, 256, 0, s, reinterpret_cast<long long*>(counts), P, (long long)(I / M) * J));
  } else {
    BIMASK_CUDA_OK(cudaMemsetAsync(counts, 0, (size_t)P * sizeof(int64_t), s));
    const int rc = M == 8 ? launch_score_m<8>(bits, cands, I, J, N, P, counts, s) : launch_score_m<16>(bits, cands, I, J, N, P, counts, s);
    if (rc != BIMASK_OK) return rc;
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

template <int M, int CRIT>
static int launch_bwd_mc(dim3 grid, int mode, const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                          int N, uint32_t* maskbits_b, uint32_t* v32, uint32_t* meta_b, const float* S, uint64_t seed,
                          uint16_t* hw16, cudaStream_t s) {
  if (mode == 1) BIMASK_CUDA_OK(launch_pdl(bwd_mask_generic_kernel<M, 1, CRIT>, grid, 256, 0, s, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16));
  else if (mode == 2) BIMASK_CUDA_OK(launch_pdl(bwd_mask_generic_kernel<M, 2, CRIT>, grid, 256, 0, s, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16));
  else BIMASK_CUDA_OK(launch_pdl(bwd_mask_generic_kernel<M, 0, CRIT>, grid, 256, 0, s, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16));
  return BIMASK_OK;
}

template <int M>
static int launch_bwd_m(int crit, dim3 grid, int mode, const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I,
                         int J, int N, uint32_t* maskbits_b, uint32_t* v32, uint32_t* meta_b, const float* S, uint64_t seed,
                         uint16_t* hw16, cudaStream_t s) {
  switch (crit) {
    case 1: return launch_bwd_mc<M, 1>(grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16, s);
    case 2: return launch_bwd_mc<M, 2>(grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16, s);
    case 3: return launch_bwd_mc<M, 3>(grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16, s);
    default: return launch_bwd_mc<M, 0>(grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b, S, seed, hw16, s);
  }
}

// criterion 0..3 as in the kernel's comment; S is read for criterion 1 only; for criterion 3 `seed`
// is hashed once here so that the per-weight key is mix64(mix64(seed) + i*J + j) >> 33.
// mode: 0 mask bits only, 1 the transposed 2:4 operand, 2 the transposed dense masked operand.
int launch_bwd_mask_criterion(const float* W, const float* S, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                              int N, int M, int crit, uint64_t seed, uint32_t* maskbits_b, uint16_t* vals_b_or_null,
                              uint32_t* meta_b_or_null, int mode, void* hw_meta_or_null, cudaStream_t s) {
  const int trip = mode == 2 ? BwdGenericTrip<2>::PASSES : BwdGenericTrip<1>::PASSES;   // 32-row passes per warp trip
  dim3 grid((I / 32 + trip - 1) / trip, (J / 32 + 7) / 8);
  uint32_t* v32 = reinterpret_cast<uint32_t*>(vals_b_or_null);
  uint16_t* hw16 = reinterpret_cast<uint16_t*>(hw_meta_or_null);
  if (crit == 3) {
    uint64_t z = seed;
    z ^= z >> 30; z *= 0xBF58476D1CE4E5B9ull; z ^= z >> 27; z *= 0x94D049BB133111EBull; z ^= z >> 31;
    seed = z;
  }
  int rc;
  if (M == 4) rc = launch_bwd_m<4>(crit, grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b_or_null, S, seed, hw16, s);
  else if (M == 8) rc = launch_bwd_m<8>(crit, grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b_or_null, S, seed, hw16, s);
  else rc = launch_bwd_m<16>(crit, grid, mode, W, maskbits_f, perm, I, J, N, maskbits_b, v32, meta_b_or_null, S, seed, hw16, s);
  if (rc != BIMASK_OK) return rc;
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

template <int N, int M>
static int refine_round(const uint32_t* bits, int32_t* perm, const int32_t* order, int I, int J, int32_t* gains,
                         unsigned long long* block_best, cudaStream_t s) {
  const int pairs = I / 2;
  BIMASK_CUDA_OK(launch_pdl(refine_gain_kernel<N, M>, (pairs + 7) / 8, 256, 0, s, bits, perm, order, I, J / 32, gains, block_best));
  BIMASK_CUDA_OK(launch_pdl(refine_apply_kernel<M>, (pairs + 255) / 256, 256, 0, s, order, gains, block_best, I, perm));
  return BIMASK_OK;
}

// rounds of greedy pairwise swaps on perm (in place).  orders: rounds x I position permutations; scratch:
// gains (I / 2 ints) and block_best (I / M 64-bit words, zeroed here before every round).
int launch_refine(const uint32_t* bits, int I, int J, int N, int M, int rounds, const int32_t* orders, int32_t* perm,
                  int32_t* gains, unsigned long long* block_best, cudaStream_t s) {
  for (int r = 0; r < rounds; ++r) {
    BIMASK_CUDA_OK(cudaMemsetAsync(block_best, 0, (size_t)(I / M) * sizeof(unsigned long long), s));
    const int32_t* order = orders + (size_t)r * I;
    int rc;
    if (M == 4) {
      if (N == 1) rc = refine_round<1, 4>(bits, perm, order, I, J, gains, block_best, s);
      else rc = refine_round<2, 4>(bits, perm, order, I, J, gains, block_best, s);
    } else if (M == 8) {
      switch (N) {
        case 1: rc = refine_round<1, 8>(bits, perm, order, I, J, gains, block_best, s); break;
        case 2: rc = refine_round<2, 8>(bits, perm, order, I, J, gains, block_best, s); break;
        case 3: rc = refine_round<3, 8>(bits, perm, order, I, J, gains, block_best, s); break;
        default: rc = refine_round<4, 8>(bits, perm, order, I, J, gains, block_best, s); break;
      }
    } else {
      switch (N) {
        case 1: rc = refine_round<1, 16>(bits, perm, order, I, J, gains, block_best, s); break;
        case 2: rc = refine_round<2, 16>(bits, perm, order, I, J, gains, block_best, s); break;
        case 3: rc = refine_round<3, 16>(bits, perm, order, I, J, gains, block_best, s); break;
        default: rc = refine_round<4, 16>(bits, perm, order, I, J, gains, block_best, s); break;
      }
    }
    if (rc != BIMASK_OK) return rc;
    count_launch();
    count_launch();
    BIMASK_CUDA_OK(cudaGetLastError());
  }
  return BIMASK_OK;
}

int launch_bwd_mask_generic(const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J, int N, int M,
                            uint32_t* maskbits_b, uint16_t* vals_b_or_null, uint32_t* meta_b_or_null, int mode,
                            void* hw_meta_or_null, cudaStream_t s) {
  return launch_bwd_mask_criterion(W, nullptr, maskbits_f, perm, I, J, N, M, 0, 0, maskbits_b, vals_b_or_null, meta_b_or_null,
                                   mode, hw_meta_or_null, s);
}

}  // namespace bimask
