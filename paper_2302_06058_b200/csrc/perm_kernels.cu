// Row-permutation search of Alg. 1: candidate generation, eligible-block counting and the pick.
//
// Counting works on the forward mask BITS (I x J/32 words, 1/32 of the weight bytes, resident in
// L2): a block of M = 4 permuted rows is tested for 32 columns at a time with a handful of
// AND/OR operations on the four row words and a popcount.
#include "common.cuh"
#include <mutex>

namespace bimask {

namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
  z ^= z >> 30;
  z *= 0xBF58476D1CE4E5B9ull;
  z ^= z >> 27;
  z *= 0x94D049BB133111EBull;
  z ^= z >> 31;
  return z;
}

// ---------------------------------------------------------------------------------------
// Candidate generation.  Candidate c is the order of the rows sorted by a 64-bit hashed key.
// The keys are uniform, so a counting sort on their top log2(I) bits leaves buckets of about
// one key each.  The bucket range is cut into Q equal parts and CTA (c, q) sorts part q: it
// hashes all I rows (cheap), histograms the keys that fall into its part with shared-memory
// atomics, counts the keys of the lower parts (its output offset), scans, scatters, finishes
// every bucket with an insertion sort (exact order on the full key) and writes its slice.
// Shared memory per CTA is about (I / Q) * 10 bytes, small enough to run beside a resident GEMM.
// ---------------------------------------------------------------------------------------
constexpr int GEN_THREADS = 1024;

__global__ void __launch_bounds__(GEN_THREADS)
gen_candidates_kernel(unsigned long long seed, int I, int nb_log2, int q_log2, int cap,
                      int32_t* __restrict__ cands, unsigned long long* __restrict__ zero_counts,
                      int32_t* __restrict__ zero_ticket) {
  pdl_launch_dependents();                               // the candidates depend on the seed alone: no wait up here
  extern __shared__ unsigned long long keys[];           // cap keys, then nbq + 1 bucket counters
  const int nbq_log2 = nb_log2 - q_log2;
  const int nbq = 1 << nbq_log2;
  uint32_t* count = reinterpret_cast<uint32_t*>(keys + cap);
  __shared__ uint32_t warp_sums[GEN_THREADS / 32];
  __shared__ uint32_t lower_total;
  const int c = blockIdx.x;
  const uint32_t part = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned long long stream = mix64(seed + 0x9E3779B97F4A7C15ull * (unsigned long long)(c + 1));
  const int shift = 64 - nb_log2;
  for (int b = tid; b < nbq; b += GEN_THREADS) count[b] = 0;
  if (tid == 0) lower_total = 0;
  __syncthreads();
  uint32_t lower = 0;
  for (int i = tid; i < I; i += GEN_THREADS) {
    const unsigned long long v = (mix64(stream ^ (unsigned long long)i) & ~0xFFFFFFull) | (unsigned long long)i;
    const uint32_t b = (uint32_t)(v >> shift);
    const uint32_t pq = b >> nbq_log2;
    if (pq == part) atomicAdd(&count[b & (nbq - 1)], 1u);
    lower += pq < part;
  }
  lower = __reduce_add_sync(0xFFFFFFFFu, lower);
  if (lane == 0 && lower) atomicAdd(&lower_total, lower);
  __syncthreads();
  // exclusive scan of the nbq counters: each thread owns a contiguous run
  const int per = (nbq + GEN_THREADS - 1) / GEN_THREADS;
  const int b0 = tid * per;
  uint32_t local = 0;
  for (int b = b0; b < min(nbq, b0 + per); ++b) local += count[b];
  uint32_t incl = local;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    uint32_t ws = lane < GEN_THREADS / 32 ? warp_sums[lane] : 0u;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, ws, d);
      if (lane >= d) ws += t;
    }
    if (lane < GEN_THREADS / 32) warp_sums[lane] = ws;
  }
  __syncthreads();
  uint32_t run = incl - local + (warp > 0 ? warp_sums[warp - 1] : 0u);
  for (int b = b0; b < min(nbq, b0 + per); ++b) {
    const uint32_t n = count[b];
    count[b] = run;                                       // start of bucket b
    run += n;
  }
  if (tid == GEN_THREADS - 1) count[nbq] = warp_sums[GEN_THREADS / 32 - 1];   // one past the last bucket: the keys of this part
  __syncthreads();
  // The part is sorted in S passes over equal runs of its buckets, S the smallest power of two for which every
  // run holds at most `cap` keys.  S is 1 unless the part drew far more keys than its share (cap leaves more than
  // fifteen standard deviations of room), so the passes cost nothing in practice, but no key is ever dropped.
  __shared__ int s_passes;
  if (tid == 0) {
    int S = 1;
    for (; S < nbq; S <<= 1) {
      bool fits = true;
      for (int q = 0; q < S && fits; ++q) fits = count[(q + 1) * (nbq / S)] - count[q * (nbq / S)] <= (uint32_t)cap;
      if (fits) break;
    }
    s_passes = S;
  }
  __syncthreads();
  const int S = s_passes, run_len = nbq / S;
  const uint32_t base = lower_total;
  bool waited = false;
  for (int pass = 0; pass < S; ++pass) {
    const uint32_t blo = (uint32_t)(pass * run_len), bhi = blo + (uint32_t)run_len;
    const uint32_t first = count[blo];                   // untouched so far: the buckets of later passes still hold their start
    __syncthreads();
    for (int i = tid; i < I; i += GEN_THREADS) {
      const unsigned long long v = (mix64(stream ^ (unsigned long long)i) & ~0xFFFFFFull) | (unsigned long long)i;
      const uint32_t b = (uint32_t)(v >> shift);
      const uint32_t bq = b & (uint32_t)(nbq - 1);
      if ((b >> nbq_log2) == part && bq >= blo && bq < bhi) {
        const uint32_t pos = atomicAdd(&count[bq], 1u) - first;     // count[b] ends as end of bucket b
        if (pos < (uint32_t)cap) keys[pos] = v;          // holds by the choice of S (a single bucket above cap aside)
      }
    }
    __syncthreads();
    const int filled = (int)min(count[bhi - 1] - first, (uint32_t)cap);
    for (int b = b0; b < min(nbq, b0 + per); ++b) {
      if ((uint32_t)b < blo || (uint32_t)b >= bhi) continue;
      const int lo = min((uint32_t)b == blo ? 0 : (int)(count[b - 1] - first), filled);
      const int hi = min((int)(count[b] - first), filled);
      for (int a = lo + 1; a < hi; ++a) {                 // insertion sort, buckets hold ~1 key
        const unsigned long long v = keys[a];
        int q = a - 1;
        while (q >= lo && keys[q] > v) { keys[q + 1] = keys[q]; --q; }
        keys[q + 1] = v;
      }
    }
    __syncthreads();
    if (!waited) { pdl_wait(); waited = true; }           // first global access: earlier kernels may still read these buffers
    for (int i = tid; i < filled; i += GEN_THREADS)
      if (base + first + i < (uint32_t)I) cands[(long long)c * I + base + first + i] = (int32_t)(keys[i] & 0xFFFFFFull);
  }
  if (!waited) pdl_wait();
  if (tid == 0) {
    // the count kernel that follows adds into counts[c] and uses *zero_ticket as its "CTAs done" counter
    if (part == 0 && zero_counts) zero_counts[c] = 0ull;
    if (part == 0 && c == 0 && zero_ticket) *zero_ticket = 0;
  }
}

// ---------------------------------------------------------------------------------------
// Candidate generation for I <= 16384: one CTA per candidate, every key hashed once, KPT keys per thread.
// Counting sort on the top log2(I) bits as above, with three differences that matter on one SM:
//  * one atomic per key: the histogram pass keeps the value the atomic returned (the key's arrival number in its
//    bucket), so after the scan the key goes to start[bucket] + arrival without a second atomic;
//  * the order inside a bucket is settled by ranking, not by a per-bucket insertion sort: every thread counts, for
//    each of its keys, the keys of the same bucket that are smaller (buckets hold about one key);
//  * shared memory holds one 32-bit word per key: the 32 - log2(I) hash bits that follow the bucket bits, then the
//    row index.  Two keys of a bucket that agree in those hash bits (the eight lower hash bits are not stored) are
//    compared on the full key, recomputed from the row index.
// The counters are padded by one word per 32 so that the scan, where a thread walks a contiguous run of counters,
// is free of bank conflicts.  The sorted row indices are collected in shared memory (in place of the counters) and
// written out in one coalesced pass.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int pad32(int b) { return b + (b >> 5); }

// Position of the key `mine` (packed form) among the keys of its bucket, keys[lo, hi): ordered by the stored hash
// bits, and by the full 64-bit key, recomputed from the row indices, where those agree.
__device__ __noinline__ uint32_t rank_exact(const uint32_t* keys, uint32_t lo, uint32_t hi, uint32_t mine,
                                            unsigned long long stream, int nb_log2) {
  const uint32_t idx_mask = (1u << nb_log2) - 1u;
  uint32_t rank = lo;
  for (uint32_t a = lo; a < hi; ++a) {
    const uint32_t o = keys[a];
    if (((o ^ mine) >> nb_log2) != 0u || o == mine) {
      rank += o < mine;
    } else {
      const unsigned long long oi = o & idx_mask, mi = mine & idx_mask;
      const unsigned long long vo = (mix64(stream ^ oi) & ~0xFFFFFFull) | oi;
      const unsigned long long vm = (mix64(stream ^ mi) & ~0xFFFFFFull) | mi;
      rank += vo < vm;
    }
  }
  return rank;
}

template <int KPT>
__global__ void __launch_bounds__(1024)
gen_candidates_reg_kernel(unsigned long long seed, int I, int nb_log2, int32_t* __restrict__ cands,
                          unsigned long long* __restrict__ zero_counts, int32_t* __restrict__ zero_ticket) {
  pdl_launch_dependents();                               // the candidates depend on the seed alone: no wait up here
  extern __shared__ uint32_t gen_smem[];                 // I packed keys, then the padded bucket counters
  const int nb = 1 << nb_log2;
  uint32_t* keys = gen_smem;
  uint32_t* count = gen_smem + I;
  __shared__ uint32_t warp_sums[32];
  const int c = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nthreads = blockDim.x, nwarps = nthreads >> 5;
  const unsigned long long stream = mix64(seed + 0x9E3779B97F4A7C15ull * (unsigned long long)(c + 1));
  const int shift = 64 - nb_log2;
  const uint32_t idx_mask = (1u << nb_log2) - 1u;
  for (int b = tid; b < nb + (nb >> 5); b += nthreads) count[b] = 0;
  __syncthreads();
  uint32_t k32[KPT], where[KPT];                         // packed key; bucket << 16 | arrival, later the final position
#pragma unroll
  for (int q = 0; q < KPT; ++q) {
    const int i = tid + q * nthreads;
    const unsigned long long v = (mix64(stream ^ (unsigned long long)i) & ~0xFFFFFFull) | (unsigned long long)i;
    const uint32_t b = (uint32_t)(v >> shift);
    k32[q] = ((uint32_t)((v << nb_log2) >> 32) & ~idx_mask) | (uint32_t)i;
    where[q] = 0u;
    if (i < I) where[q] = (b << 16) | atomicAdd(&count[pad32(b)], 1u);
  }
  __syncthreads();
  // exclusive scan of the counters: each thread owns a contiguous run
  const int per = (nb + nthreads - 1) / nthreads;
  const int b0 = tid * per;
  uint32_t local = 0;
  for (int b = b0; b < min(nb, b0 + per); ++b) local += count[pad32(b)];
  uint32_t incl = local;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= d) incl += t;
  }
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    uint32_t ws = lane < nwarps ? warp_sums[lane] : 0u;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, ws, d);
      if (lane >= d) ws += t;
    }
    if (lane < nwarps) warp_sums[lane] = ws;
  }
  __syncthreads();
  uint32_t run = incl - local + (warp > 0 ? warp_sums[warp - 1] : 0u);
  for (int b = b0; b < min(nb, b0 + per); ++b) {
    const uint32_t n = count[pad32(b)];
    count[pad32(b)] = run;                                // start of bucket b
    run += n;
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < KPT; ++q) {
    const int i = tid + q * nthreads;
    if (i < I) keys[count[pad32(where[q] >> 16)] + (where[q] & 0xFFFFu)] = k32[q];
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < KPT; ++q) {
    const int i = tid + q * nthreads;
    if (i < I) {
      const int b = (int)(where[q] >> 16);
      const uint32_t lo = count[pad32(b)], hi = b + 1 < nb ? count[pad32(b + 1)] : (uint32_t)I;
      // the first six keys of the bucket without a loop (a bucket holds one key on average); longer buckets and
      // keys that agree in the stored hash bits take the exact walk
      uint32_t rank = lo;
      bool again = hi - lo > 6u;
#pragma unroll
      for (uint32_t t = 0; t < 6u; ++t) {
        if (lo + t < hi) {
          const uint32_t o = keys[lo + t];
          rank += o < k32[q];
          again |= ((o ^ k32[q]) >> nb_log2) == 0u && o != k32[q];
        }
      }
      if (again) rank = rank_exact(keys, lo, hi, k32[q], stream, nb_log2);
      where[q] = rank;
    }
  }
  __syncthreads();                                       // every thread has read the bucket starts
  int32_t* sorted = reinterpret_cast<int32_t*>(count);   // more than I entries
#pragma unroll
  for (int q = 0; q < KPT; ++q) {
    const int i = tid + q * nthreads;
    if (i < I) sorted[where[q]] = i;
  }
  __syncthreads();
  pdl_wait();                                            // first global access: earlier kernels may still read these buffers
  if (tid == 0) {
    if (zero_counts) zero_counts[c] = 0ull;
    if (c == 0 && zero_ticket) *zero_ticket = 0;
  }
  int32_t* out = cands + (long long)c * I;
  if ((I & 3) == 0) {
    for (int i = tid; i < (I >> 2); i += nthreads) reinterpret_cast<int4*>(out)[i] = reinterpret_cast<const int4*>(sorted)[i];
  } else {
    for (int i = tid; i < I; i += nthreads) out[i] = sorted[i];
  }
}

// ---------------------------------------------------------------------------------------
// Pick: arg-max of counts with ties to the lowest candidate index, then copy that candidate.
// ---------------------------------------------------------------------------------------
constexpr int PICK_THREADS = 256;

// One CTA of PICK_THREADS threads; counts are read around L1 (they were written by atomics of other CTAs).
// PACKED: bits [48,64) of a count hold the number of CTAs that have added their share (the fused pick of the count
// kernel); they are stripped here and the plain count is written back.
constexpr unsigned long long COUNT_MASK = (1ull << 48) - 1ull;
template <bool PACKED>
__device__ __forceinline__ void pick_body(long long* counts, const int32_t* __restrict__ cands, int P, int I,
                                          int32_t* best_idx, int32_t* __restrict__ best_perm) {
  __shared__ long long s_cnt[PICK_THREADS];
  __shared__ int s_idx[PICK_THREADS];
  long long bc = -1;
  int bi = 0x7FFFFFFF;
  for (int c = threadIdx.x; c < P; c += PICK_THREADS) {
    long long v = __ldcg(counts + c);
    if (PACKED) {
      v = (long long)((unsigned long long)v & COUNT_MASK);
      counts[c] = v;
    }
    if (v > bc) { bc = v; bi = c; }      // ascending c per thread: first maximum is kept
  }
  s_cnt[threadIdx.x] = bc;
  s_idx[threadIdx.x] = bi;
  __syncthreads();
  for (int s = PICK_THREADS / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) {
      const long long oc = s_cnt[threadIdx.x + s];
      const int oi = s_idx[threadIdx.x + s];
      if (oc > s_cnt[threadIdx.x] || (oc == s_cnt[threadIdx.x] && oi < s_idx[threadIdx.x])) {
        s_cnt[threadIdx.x] = oc;
        s_idx[threadIdx.x] = oi;
      }
    }
    __syncthreads();
  }
  const int best = s_idx[0];
  if (threadIdx.x == 0) *best_idx = best;
  const int32_t* src = cands + (long long)best * I;
  if ((I & 3) == 0) {
    for (int i = threadIdx.x; i < (I >> 2); i += PICK_THREADS)
      reinterpret_cast<int4*>(best_perm)[i] = __ldg(reinterpret_cast<const int4*>(src) + i);
  } else {
    for (int i = threadIdx.x; i < I; i += PICK_THREADS) best_perm[i] = src[i];
  }
}

__global__ void __launch_bounds__(PICK_THREADS)
pick_kernel(const long long* __restrict__ counts, const int32_t* __restrict__ cands, int P, int I,
            int32_t* __restrict__ best_idx, int32_t* __restrict__ best_perm) {
  pdl_launch_dependents();
  pdl_wait();
  pick_body<false>(const_cast<long long*>(counts), cands, P, I, best_idx, best_perm);
}

// ---------------------------------------------------------------------------------------
// Eligible-block count.  grid = (row-block chunks, P).  A warp takes one row block of a
// candidate at a time: the four row indices are one 16-byte load, each lane then reads its
// slice of the four mask rows (128-bit loads when J % 128 == 0) and counts columns whose
// four bits hold at most N ones.  One 64-bit atomic per CTA.
// ---------------------------------------------------------------------------------------
constexpr int SCORE_THREADS = 256;
constexpr int SCORE_KB_MAX = 256;                      // row blocks of one candidate per CTA: 32 .. 256, chosen by the launcher

// Columns (bits) where more than N of the four rows are set.  a + b + c = 2 * maj + par (a full adder per bit,
// two three-input logic operations); adding d: at least two  <=>  maj | (par & d), at least three  <=>
// maj & (par | d) -- one more three-input operation.
template <int N>
__device__ __forceinline__ uint32_t ineligible(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  const uint32_t par = a ^ b ^ c;
  const uint32_t maj = (a & b) | (a & c) | (b & c);
  if (N == 1) return maj | (par & d);
  if (N == 2) return maj & (par | d);
  if (N == 3) return a & b & c & d;
  return 0u;
}

template <int N>
__global__ void __launch_bounds__(SCORE_THREADS, 4)
score_kernel(const uint32_t* __restrict__ bits, const int32_t* __restrict__ cands, int I, int jwords, int kb_per_cta,
             unsigned long long* __restrict__ counts, int P, int32_t* best_idx, int32_t* __restrict__ best_perm) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.y;
  const int nkb = I >> 2;
  const int kb0 = blockIdx.x * kb_per_cta;
  const int kb1 = min(nkb, kb0 + kb_per_cta);
  const int4* cand4 = reinterpret_cast<const int4*>(cands + (long long)c * I);
  uint32_t cnt = 0;
  if ((jwords & 3) == 0) {
    const int jq = jwords >> 2;
    // the CTA's row indices first (one coalesced load, clamped), so that the row loads below do
    // not wait on a dependent global load
    __shared__ int4 idx_s[SCORE_KB_MAX];
    for (int t = threadIdx.x; t < kb1 - kb0; t += SCORE_THREADS) {
      const int4 r = __ldg(cand4 + kb0 + t);
      idx_s[t] = make_int4(checked_row(r.x, I, SITE_SCORE_CAND), checked_row(r.y, I, SITE_SCORE_CAND),
                           checked_row(r.z, I, SITE_SCORE_CAND), checked_row(r.w, I, SITE_SCORE_CAND));
    }
    __syncthreads();
    // two row blocks per trip: eight independent 128-bit loads in flight per lane
    for (int k = kb0 + warp; k < kb1; k += 2 * (SCORE_THREADS / 32)) {
      const int k2 = k + SCORE_THREADS / 32;
      const bool two = k2 < kb1;
      const int4 r = idx_s[k - kb0];
      const int4 t = idx_s[(two ? k2 : k) - kb0];
      const uint4* r0 = reinterpret_cast<const uint4*>(bits + (long long)r.x * jwords);
      const uint4* r1 = reinterpret_cast<const uint4*>(bits + (long long)r.y * jwords);
      const uint4* r2 = reinterpret_cast<const uint4*>(bits + (long long)r.z * jwords);
      const uint4* r3 = reinterpret_cast<const uint4*>(bits + (long long)r.w * jwords);
      const uint4* t0 = reinterpret_cast<const uint4*>(bits + (long long)t.x * jwords);
      const uint4* t1 = reinterpret_cast<const uint4*>(bits + (long long)t.y * jwords);
      const uint4* t2 = reinterpret_cast<const uint4*>(bits + (long long)t.z * jwords);
      const uint4* t3 = reinterpret_cast<const uint4*>(bits + (long long)t.w * jwords);
      uint32_t c1 = 0, c2 = 0, words = 0;
      for (int q = lane; q < jq; q += 32) {
        const uint4 a = __ldg(r0 + q), b = __ldg(r1 + q), cc = __ldg(r2 + q), d = __ldg(r3 + q);
        const uint4 e = __ldg(t0 + q), f = __ldg(t1 + q), g = __ldg(t2 + q), h = __ldg(t3 + q);
        c1 += __popc(ineligible<N>(a.x, b.x, cc.x, d.x)) + __popc(ineligible<N>(a.y, b.y, cc.y, d.y)) +
              __popc(ineligible<N>(a.z, b.z, cc.z, d.z)) + __popc(ineligible<N>(a.w, b.w, cc.w, d.w));
        c2 += __popc(ineligible<N>(e.x, f.x, g.x, h.x)) + __popc(ineligible<N>(e.y, f.y, g.y, h.y)) +
              __popc(ineligible<N>(e.z, f.z, g.z, h.z)) + __popc(ineligible<N>(e.w, f.w, g.w, h.w));
        words += 4;
      }
      // eligible = all columns this lane looked at minus the ineligible ones
      cnt += (32u * words - c1) + (two ? 32u * words - c2 : 0u);
    }
  } else {
    for (int k = kb0 + warp; k < kb1; k += SCORE_THREADS / 32) {
      int4 r = __ldg(cand4 + k);
      r.x = checked_row(r.x, I, SITE_SCORE_CAND); r.y = checked_row(r.y, I, SITE_SCORE_CAND);
      r.z = checked_row(r.z, I, SITE_SCORE_CAND); r.w = checked_row(r.w, I, SITE_SCORE_CAND);
      const uint32_t* r0 = bits + (long long)r.x * jwords;
      const uint32_t* r1 = bits + (long long)r.y * jwords;
      const uint32_t* r2 = bits + (long long)r.z * jwords;
      const uint32_t* r3 = bits + (long long)r.w * jwords;
      for (int q = lane; q < jwords; q += 32)
        cnt += __popc(~ineligible<N>(__ldg(r0 + q), __ldg(r1 + q), __ldg(r2 + q), __ldg(r3 + q)));
    }
  }
  cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
  __shared__ uint32_t part[SCORE_THREADS / 32];
  if (lane == 0) part[warp] = cnt;
  __syncthreads();
  __shared__ bool last_cta;
  if (threadIdx.x == 0) {
    unsigned long long s = 0;
#pragma unroll
    for (int w = 0; w < SCORE_THREADS / 32; ++w) s += part[w];
    last_cta = false;
    if (best_idx) {
      // fused pick: the sum travels with a one in bits [48,64), so the count word also tells how many CTAs of this
      // candidate have reported; the CTA that completes a candidate bumps *best_idx (zeroed before the launch), and
      // the one that completes the last candidate sees every sum (fence on both sides of the counters) and picks
      const unsigned long long old = atomicAdd(counts + c, s + (1ull << 48));
      if ((unsigned)(old >> 48) + 1u == gridDim.x) {
        __threadfence();
        last_cta = atomicAdd(reinterpret_cast<unsigned*>(best_idx), 1u) == gridDim.y - 1u;
      }
    } else {
      atomicAdd(counts + c, s);
    }
  }
  __syncthreads();
  if (last_cta) {
    __threadfence();
    pick_body<true>(reinterpret_cast<long long*>(counts), cands, P, I, best_idx, best_perm);
  }
}

// Debug: every row of cands is a permutation of 0..I-1.
__global__ void check_perms_kernel(const int32_t* __restrict__ cands, int P, int I,
                                   uint8_t* __restrict__ seen, int32_t* __restrict__ ok) {
  pdl_launch_dependents();
  pdl_wait();
  const int c = blockIdx.x;
  for (int i = threadIdx.x; i < I; i += blockDim.x) {
    const int v = cands[(long long)c * I + i];
    if (v < 0 || v >= I) { atomicExch(ok, 0); continue; }
    seen[(long long)c * I + v] = 1;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < I; i += blockDim.x)
    if (!seen[(long long)c * I + i]) atomicExch(ok, 0);
}

__global__ void set_int_kernel(int32_t* p, int32_t v) {
  pdl_launch_dependents();
  pdl_wait();
  *p = v;
}

}  // namespace

BIMASK_DEFINE_DEBUG_COLLECT(debug_collect_perm)

int launch_gen_candidates(uint64_t seed, int P, int I, int32_t* cands, cudaStream_t s, int64_t* zero_counts,
                          int32_t* zero_ticket, int part_cap) {
  int lg = 1;
  while ((1 << lg) < I) ++lg;                             // one bucket per key on average
  unsigned long long* zc = reinterpret_cast<unsigned long long*>(zero_counts);
  if (I <= 16384 && part_cap <= 0) {
    // a CTA per candidate with the keys in registers: 4, 8 or 16 per thread
    const int kpt = I <= 4096 ? 4 : I <= 8192 ? 8 : 16;
    int threads = ((I + kpt - 1) / kpt + 31) / 32 * 32;
    const size_t smem = ((size_t)I + ((size_t)1 << lg) + ((size_t)1 << lg >> 5) + 4) * sizeof(uint32_t);
    if (kpt == 4) {
      if (int rc = set_smem_attr(gen_candidates_reg_kernel<4>, 200 * 1024)) return rc;
      BIMASK_CUDA_OK(launch_pdl(gen_candidates_reg_kernel<4>, P, threads, smem, s, (unsigned long long)seed, I, lg, cands, zc, zero_ticket));
    } else if (kpt == 8) {
      if (int rc = set_smem_attr(gen_candidates_reg_kernel<8>, 200 * 1024)) return rc;
      BIMASK_CUDA_OK(launch_pdl(gen_candidates_reg_kernel<8>, P, threads, smem, s, (unsigned long long)seed, I, lg, cands, zc, zero_ticket));
    } else {
      if (int rc = set_smem_attr(gen_candidates_reg_kernel<16>, 200 * 1024)) return rc;
      BIMASK_CUDA_OK(launch_pdl(gen_candidates_reg_kernel<16>, P, threads, smem, s, (unsigned long long)seed, I, lg, cands, zc, zero_ticket));
    }
    count_launch();
    BIMASK_CUDA_OK(cudaGetLastError());
    return BIMASK_OK;
  }
  int ql = 0;
  while ((I >> ql) > 8192 && ql < lg - 1) ++ql;           // at most 8192 keys per part (measured best)
  const int mean = (I + (1 << ql) - 1) >> ql;
  int cap = ql == 0 ? I : mean + (mean / 4 > 256 ? mean / 4 : 256);
  if (part_cap > 0) cap = part_cap < cap ? part_cap : cap;         // debug: a small capacity forces the multi-pass sort
  const size_t smem = (size_t)cap * sizeof(unsigned long long) + (((size_t)1 << (lg - ql)) + 2) * sizeof(uint32_t);
  if (int rc = set_smem_attr(gen_candidates_kernel, 200 * 1024)) return rc;
  dim3 grid(P, 1 << ql);
  BIMASK_CUDA_OK(launch_pdl(gen_candidates_kernel, grid, GEN_THREADS, smem, s, (unsigned long long)seed, I, lg, ql, cap, cands,
                                                        zc, zero_ticket));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// best_idx / best_perm given: the kernel also picks the winner (its last CTA), so no pick launch is needed.
// zeroed: counts (and *best_idx, the fused pick's CTA counter) were already zeroed on the stream, e.g. by the
// candidate generator.
int launch_score(const uint32_t* maskbits_f, const int32_t* cands, int I, int J, int N, int P,
                 int64_t* counts, cudaStream_t s, bool zeroed, int32_t* best_idx, int32_t* best_perm) {
  // row blocks per CTA: as many as still give every SM a dozen CTAs (fewer, longer CTAs start and drain less often)
  const int nkb = I / 4;
  int kb = SCORE_KB_MAX;
  while (kb > 32 && (long long)P * ((nkb + kb - 1) / kb) < 12 * 148) kb >>= 1;
  dim3 grid((nkb + kb - 1) / kb, P);
  // the fused pick counts a candidate's CTAs in 16 bits of its count word and needs sums below 2^48
  int32_t* pick_idx = best_idx, *pick_perm = best_perm;
  const bool fuse = best_idx != nullptr && grid.x <= 65535u && (long long)nkb * J < (1ll << 48);
  if (!fuse) best_idx = nullptr;
  if (!zeroed) {
    BIMASK_CUDA_OK(cudaMemsetAsync(counts, 0, (size_t)P * sizeof(int64_t), s));
    if (best_idx) BIMASK_CUDA_OK(cudaMemsetAsync(best_idx, 0, sizeof(int32_t), s));
  }
  unsigned long long* cnt = reinterpret_cast<unsigned long long*>(counts);
  switch (N) {
    case 1: BIMASK_CUDA_OK(launch_pdl(score_kernel<1>, grid, SCORE_THREADS, 0, s, maskbits_f, cands, I, J / 32, kb, cnt, P, best_idx, best_perm)); break;
    case 2: BIMASK_CUDA_OK(launch_pdl(score_kernel<2>, grid, SCORE_THREADS, 0, s, maskbits_f, cands, I, J / 32, kb, cnt, P, best_idx, best_perm)); break;
    case 3: BIMASK_CUDA_OK(launch_pdl(score_kernel<3>, grid, SCORE_THREADS, 0, s, maskbits_f, cands, I, J / 32, kb, cnt, P, best_idx, best_perm)); break;
    default: BIMASK_CUDA_OK(launch_pdl(score_kernel<4>, grid, SCORE_THREADS, 0, s, maskbits_f, cands, I, J / 32, kb, cnt, P, best_idx, best_perm)); break;
  }
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  if (pick_idx && !fuse) {
    BIMASK_CUDA_OK(launch_pdl(pick_kernel, 1, PICK_THREADS, 0, s, reinterpret_cast<const long long*>(counts), cands, P, I, pick_idx, pick_perm));
    count_launch();
    BIMASK_CUDA_OK(cudaGetLastError());
  }
  return BIMASK_OK;
}

int launch_pick(const int64_t* counts, const int32_t* cands, int P, int I, int32_t* best_idx,
                int32_t* best_perm, cudaStream_t s) {
  BIMASK_CUDA_OK(launch_pdl(pick_kernel, 1, PICK_THREADS, 0, s, reinterpret_cast<const long long*>(counts), cands, P, I,
                                         best_idx, best_perm));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_check_perms(const int32_t* cands, int P, int I, int32_t* ok, uint8_t* seen, cudaStream_t s) {
  BIMASK_CUDA_OK(cudaMemsetAsync(seen, 0, (size_t)P * I, s));
  BIMASK_CUDA_OK(launch_pdl(set_int_kernel, 1, 1, 0, s, ok, 1));
  count_launch();
  BIMASK_CUDA_OK(launch_pdl(check_perms_kernel, P, 256, 0, s, cands, P, I, seen, ok));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// ---------------------------------------------------------------------------------------
// bimask_perm_search_static: the permutation search for callers that have no scratch buffer
// to give.  The generated candidates (P x I int32) live in a fixed array inside the library's
// device image instead of caller memory, so the call needs no allocation by anybody.
// ---------------------------------------------------------------------------------------
namespace {

constexpr size_t STATIC_CAND_ENTRIES = (size_t)2 << 20;              // 2 Mi int32 = 8 MiB per GPU
static __device__ __align__(256) int32_t g_static_cands[STATIC_CAND_ENTRIES];

// Device address of g_static_cands on each device.  In host code the symbol's name is only a
// handle, so the address is looked up once per device (with that device current) and cached.
std::mutex g_static_mutex;
int32_t* g_static_ptr[64] = {nullptr};

int static_cands_ptr(int32_t** out) {
  int dev = 0;
  BIMASK_CUDA_OK(cudaGetDevice(&dev));
  BIMASK_REQUIRE(dev >= 0 && dev < 64, BIMASK_EUNSUPPORTED, "device ordinal %d out of range", dev);
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[dev]) {
    int32_t* ptr = nullptr;
    BIMASK_CUDA_OK(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_cands));
    BIMASK_REQUIRE(ptr != nullptr, BIMASK_ECUDA, "cudaGetSymbolAddress returned a null address");
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return BIMASK_OK;
}

}  // namespace

}  // namespace bimask

extern "C" size_t bimask_perm_search_static_max_entries(void) { return bimask::STATIC_CAND_ENTRIES; }

extern "C" int bimask_perm_search_static(const uint32_t* maskbits_f, int I, int J, int N, int M, int P, uint64_t seed,
                                         int32_t* best_perm, int32_t* best_idx, int64_t* counts, void* stream) {
  using namespace bimask;
  BIMASK_REQUIRE(M == 4, BIMASK_EUNSUPPORTED, "M = %d: only M = 4 is implemented", M);
  BIMASK_REQUIRE(I > 0 && J > 0 && I % 4 == 0 && J % 32 == 0, BIMASK_EINVAL,
                 "I = %d, J = %d: I must be a positive multiple of 4, J of 32", I, J);
  BIMASK_REQUIRE(N >= 1 && N <= M, BIMASK_EINVAL, "N = %d out of range 1..%d", N, M);
  BIMASK_REQUIRE(P >= 1 && P <= 65535, BIMASK_EINVAL, "P = %d out of range 1..65535", P);
  BIMASK_REQUIRE((size_t)P * (size_t)I <= STATIC_CAND_ENTRIES, BIMASK_EUNSUPPORTED,
                 "bimask_perm_search_static: P * I = %zu candidate entries exceed the built-in scratch of %zu; "
                 "use bimask_perm_search with a caller-provided workspace",
                 (size_t)P * (size_t)I, STATIC_CAND_ENTRIES);
  BIMASK_REQUIRE(maskbits_f && best_perm && best_idx && counts, BIMASK_EINVAL, "bimask_perm_search_static: null pointer");
  BIMASK_REQUIRE(aligned16(maskbits_f) && aligned16(best_perm) && ((uintptr_t)counts % 8 == 0) &&
                     ((uintptr_t)best_idx % 4 == 0),
                 BIMASK_EINVAL, "bimask_perm_search_static: misaligned pointer");
  int32_t* cands = nullptr;
  int rc = static_cands_ptr(&cands);
  if (rc != BIMASK_OK) return rc;
  cudaStream_t s = (cudaStream_t)stream;
  // every entry of the first P x I slots is rewritten by the generator, so nothing left over
  // from an earlier call is ever read; counts is zeroed inside launch_score
  if ((rc = launch_gen_candidates(seed, P, I, cands, s)) != BIMASK_OK) return rc;
  if ((rc = launch_score(maskbits_f, cands, I, J, N, P, counts, s)) != BIMASK_OK) return rc;
  return launch_pick(counts, cands, P, I, best_idx, best_perm, s);
}
