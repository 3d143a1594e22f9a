// C ABI of the library: argument validation, workspace carving and the order of launches.
// No kernel code lives here.
#include "common.cuh"
#include <string.h>
#include <atomic>
#include <mutex>

namespace bimask {

static thread_local char g_err[512] = "";
static std::atomic<unsigned long long> g_launches{0};

void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

int cuda_fail(cudaError_t e, const char* what) {
  set_error("%s failed: %s", what, cudaGetErrorString(e));
  return BIMASK_ECUDA;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Shapes and pattern of the mask calls.  *pack: the pattern fits the 2:4 container (N <= 2).
static int check_shape(int I, int J, int N, int M, bool* pack) {
  BIMASK_REQUIRE(M == 4 || M == 8 || M == 16, BIMASK_EUNSUPPORTED, "M = %d: block lengths 4, 8 and 16 are implemented", M);
  BIMASK_REQUIRE(I > 0 && J > 0 && I % 32 == 0 && J % 32 == 0, BIMASK_EINVAL,
                 "I = %d, J = %d: both must be positive multiples of 32", I, J);
  BIMASK_REQUIRE(N >= 1 && N <= M, BIMASK_EINVAL, "N = %d out of range 1..%d", N, M);
  BIMASK_REQUIRE(M != 4 || N <= 2, BIMASK_EUNSUPPORTED, "N:M = %d:%d does not fit the 2:4 container", N, M);
  *pack = N <= 2;
  return BIMASK_OK;
}

struct WsPlan {
  size_t cands_off, cands_bytes;
  size_t dyp_off, dyp_bytes;
  size_t part_off, part_bytes;
  size_t total;
};

static WsPlan plan_ws(int T, int I, int J, int P) {
  WsPlan w;
  size_t off = 0;
  w.cands_off = off; w.cands_bytes = align_up((size_t)(P > 0 ? P : 0) * I * sizeof(int32_t), 256); off += w.cands_bytes;
  w.dyp_off = off; w.dyp_bytes = align_up((size_t)(T > 0 ? T : 0) * I * 2, 256); off += w.dyp_bytes;
  int nt = 0, splits = 1, per = 0;
  if (T > 0) wgrad_plan(T, I, J, &nt, &splits, &per);
  w.part_off = off; w.part_bytes = splits > 1 ? align_up((size_t)splits * I * J * sizeof(float), 256) : 0; off += w.part_bytes;
  w.total = off > 256 ? off : 256;
  return w;
}

}  // namespace bimask

using namespace bimask;

extern "C" {

const char* bimask_last_error(void) { return g_err; }

uint64_t bimask_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t bimask_hw_meta_bytes(int rows, int K) {
  if (rows <= 0 || K <= 0) return 0;
  return (size_t)((rows + 127) / 128) * ((K + 127) / 128) * 2048;
}

size_t bimask_workspace_bytes(int T, int I, int J, int P) {
  if (I <= 0 || J <= 0) return 0;
  return plan_ws(T, I, J, P).total;
}

int bimask_fwd_mask(const float* W, int I, int J, int N, int M, uint32_t* maskbits_f, uint16_t* vals_f,
                    uint32_t* meta_f, void* hw_meta_f, void* stream) {
  bool pack = false;
  int rc = check_shape(I, J, N, M, &pack);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(W && maskbits_f, BIMASK_EINVAL, "bimask_fwd_mask: null pointer");
  if (pack) {
    BIMASK_REQUIRE(vals_f && meta_f && hw_meta_f, BIMASK_EINVAL, "bimask_fwd_mask: null pointer");
  } else {
    BIMASK_REQUIRE(!meta_f && !hw_meta_f, BIMASK_EUNSUPPORTED,
                   "N:M = %d:%d does not fit the 2:4 container: pass meta_f = hw_meta_f = NULL (vals_f, when given, receives the "
                   "dense masked operand)",
                   N, M);
  }
  BIMASK_REQUIRE(aligned16(W) && aligned16(maskbits_f) && aligned16(vals_f) && aligned16(meta_f) && aligned16(hw_meta_f),
                 BIMASK_EINVAL, "bimask_fwd_mask: pointers must be 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  if (M != 4) {
    const bool gfused = pack && (I % 128 == 0) && (J % 128 == 0);   // unpadded: the mask kernel writes the metadata image
    if ((rc = launch_fwd_mask_generic(W, I, J, N, M, maskbits_f, vals_f, meta_f, pack ? 1 : vals_f ? 2 : 0,
                                      gfused ? hw_meta_f : nullptr, s)) != BIMASK_OK)
      return rc;
    return pack && !gfused ? launch_hw_meta(meta_f, I, J, hw_meta_f, s) : BIMASK_OK;
  }
  return launch_fwd_mask(W, I, J, N, maskbits_f, vals_f, meta_f, hw_meta_f, s);   // writes the metadata image too, padding included
}

size_t bimask_refine_workspace_bytes(int I, int M, int rounds) {
  if (I <= 0 || rounds < 0 || (M != 4 && M != 8 && M != 16)) return 0;
  return align_up((size_t)rounds * I * sizeof(int32_t), 256) + align_up((size_t)(I / 2) * sizeof(int32_t), 256) +
         align_up((size_t)(I / M) * sizeof(unsigned long long), 256);
}

int bimask_perm_refine(const uint32_t* maskbits_f, int I, int J, int N, int M, int rounds, uint64_t seed,
                       int32_t* perm_inout, int64_t* count_out, void* ws, size_t ws_bytes, void* stream) {
  BIMASK_REQUIRE(M == 4 || M == 8 || M == 16, BIMASK_EUNSUPPORTED, "M = %d: block lengths 4, 8 and 16 are implemented", M);
  BIMASK_REQUIRE(I > 0 && J > 0 && I % M == 0 && I % 2 == 0 && J % 32 == 0, BIMASK_EINVAL,
                 "I = %d, J = %d: I must be a positive even multiple of M, J of 32", I, J);
  BIMASK_REQUIRE(N >= 1 && N <= M, BIMASK_EINVAL, "N = %d out of range 1..%d", N, M);
  BIMASK_REQUIRE(N <= 4 && (M != 4 || N <= 2), BIMASK_EUNSUPPORTED, "N:M = %d:%d: the refinement counts blocks for N <= 4 (N <= 2 at M = 4)", N, M);
  BIMASK_REQUIRE(rounds >= 0 && rounds <= 4096, BIMASK_EINVAL, "rounds = %d out of range 0..4096", rounds);
  BIMASK_REQUIRE(I < (1 << 24), BIMASK_EUNSUPPORTED, "the pairing generator needs I < 2^24 (I = %d)", I);
  BIMASK_REQUIRE(maskbits_f && perm_inout && ws, BIMASK_EINVAL, "bimask_perm_refine: null pointer");
  BIMASK_REQUIRE(aligned16(maskbits_f) && aligned16(perm_inout) && aligned16(ws) && (!count_out || (uintptr_t)count_out % 8 == 0),
                 BIMASK_EINVAL, "bimask_perm_refine: misaligned pointer");
  const size_t need = bimask_refine_workspace_bytes(I, M, rounds);
  BIMASK_REQUIRE(ws_bytes >= need, BIMASK_EINVAL, "bimask_perm_refine: workspace too small (%zu bytes, need %zu)", ws_bytes, need);
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* w8 = reinterpret_cast<uint8_t*>(ws);
  int32_t* orders = reinterpret_cast<int32_t*>(w8);
  int32_t* gains = reinterpret_cast<int32_t*>(w8 + align_up((size_t)rounds * I * sizeof(int32_t), 256));
  unsigned long long* best = reinterpret_cast<unsigned long long*>(reinterpret_cast<uint8_t*>(gains) +
                                                                   align_up((size_t)(I / 2) * sizeof(int32_t), 256));
  int rc;
  if (rounds > 0) {
    // the random pairings of all rounds: `rounds` permutations of the positions, same generator as the candidates
    if ((rc = launch_gen_candidates(seed + 0x5EED5EEDull, rounds, I, orders, s)) != BIMASK_OK) return rc;
    if ((rc = launch_refine(maskbits_f, I, J, N, M, rounds, orders, perm_inout, gains, best, s)) != BIMASK_OK) return rc;
  }
  if (count_out) {
    if (M == 4) return launch_score(maskbits_f, perm_inout, I, J, N, 1, count_out, s);
    return launch_score_generic(maskbits_f, perm_inout, I, J, N, M, 1, count_out, s);
  }
  return BIMASK_OK;
}

int bimask_sgd_fwd_mask(float* W, const float* dW, float* mom, int I, int J, int N, int M, float lr, float momentum,
                        float weight_decay, uint32_t* maskbits_f, uint16_t* vals_f, uint32_t* meta_f, void* hw_meta_f,
                        void* stream) {
  bool pack = false;
  int rc = check_shape(I, J, N, M, &pack);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(W && dW && maskbits_f, BIMASK_EINVAL, "bimask_sgd_fwd_mask: null pointer");
  if (pack) {
    BIMASK_REQUIRE(vals_f && meta_f && hw_meta_f, BIMASK_EINVAL, "bimask_sgd_fwd_mask: null pointer");
  } else {
    BIMASK_REQUIRE(!meta_f && !hw_meta_f, BIMASK_EUNSUPPORTED,
                   "N:M = %d:%d does not fit the 2:4 container: pass meta_f = hw_meta_f = NULL (vals_f, when given, receives the "
                   "dense masked operand)",
                   N, M);
  }
  BIMASK_REQUIRE(aligned16(W) && aligned16(dW) && aligned16(mom) && aligned16(maskbits_f) && aligned16(vals_f) &&
                     aligned16(meta_f) && aligned16(hw_meta_f),
                 BIMASK_EINVAL, "bimask_sgd_fwd_mask: pointers must be 16-byte aligned");
  BIMASK_REQUIRE(lr == lr && momentum == momentum && weight_decay == weight_decay, BIMASK_EINVAL,
                 "bimask_sgd_fwd_mask: NaN hyper-parameter");
  cudaStream_t s = (cudaStream_t)stream;
  if (M != 4) {
    const bool gfused = pack && (I % 128 == 0) && (J % 128 == 0);   // unpadded: the mask kernel writes the metadata image
    if ((rc = launch_fwd_mask_generic(W, I, J, N, M, maskbits_f, vals_f, meta_f, pack ? 1 : vals_f ? 2 : 0,
                                      gfused ? hw_meta_f : nullptr, s, dW, mom, lr, momentum, weight_decay)) != BIMASK_OK)
      return rc;
    return pack && !gfused ? launch_hw_meta(meta_f, I, J, hw_meta_f, s) : BIMASK_OK;
  }
  return launch_sgd_fwd_mask(W, dW, mom, I, J, N, lr, momentum, weight_decay, maskbits_f, vals_f, meta_f, hw_meta_f, s);
}

int bimask_perm_search(const uint32_t* maskbits_f, int I, int J, int N, int M, int P, uint64_t seed,
                       const int32_t* cands_or_null, int32_t* best_perm, int32_t* best_idx, int64_t* counts,
                       void* ws, size_t ws_bytes, void* stream) {
  BIMASK_REQUIRE(M == 4 || M == 8 || M == 16, BIMASK_EUNSUPPORTED, "M = %d: block lengths 4, 8 and 16 are implemented", M);
  BIMASK_REQUIRE(I > 0 && J > 0 && I % M == 0 && J % 32 == 0, BIMASK_EINVAL,
                 "I = %d, J = %d: I must be a positive multiple of M, J of 32", I, J);
  BIMASK_REQUIRE(N >= 1 && N <= M, BIMASK_EINVAL, "N = %d out of range 1..%d", N, M);
  BIMASK_REQUIRE(M == 4 || N <= 4 || N == M, BIMASK_EUNSUPPORTED, "N:M = %d:%d: the count kernel handles N <= 4", N, M);
  BIMASK_REQUIRE(P >= 1 && P <= 65535, BIMASK_EINVAL, "P = %d out of range 1..65535", P);
  BIMASK_REQUIRE(maskbits_f && best_perm && best_idx && counts, BIMASK_EINVAL, "bimask_perm_search: null pointer");
  BIMASK_REQUIRE(aligned16(maskbits_f) && aligned16(best_perm) && (!cands_or_null || aligned16(cands_or_null)) &&
                     ((uintptr_t)counts % 8 == 0) && ((uintptr_t)best_idx % 4 == 0),
                 BIMASK_EINVAL, "bimask_perm_search: misaligned pointer");
  cudaStream_t s = (cudaStream_t)stream;
  const int32_t* cands = cands_or_null;
  int rc;
  if (!cands) {
    BIMASK_REQUIRE(I < (1 << 24), BIMASK_EUNSUPPORTED, "generated candidates need I < 2^24 (I = %d)", I);
    const WsPlan w = plan_ws(0, I, J, P);
    BIMASK_REQUIRE(ws && aligned16(ws) && ws_bytes >= w.cands_off + w.cands_bytes, BIMASK_EINVAL,
                   "bimask_perm_search: workspace too small (%zu bytes, need %zu)", ws_bytes, w.cands_off + w.cands_bytes);
    int32_t* gen = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(ws) + w.cands_off);
    // M = 4: the generator zeroes counts and the pick's CTA counter, the count kernel picks the winner itself
    if ((rc = launch_gen_candidates(seed, P, I, gen, s, M == 4 ? counts : nullptr, M == 4 ? best_idx : nullptr)) != BIMASK_OK)
      return rc;
    cands = gen;
  }
  if (M == 4) return launch_score(maskbits_f, cands, I, J, N, P, counts, s, cands_or_null == nullptr, best_idx, best_perm);
  if ((rc = launch_score_generic(maskbits_f, cands, I, J, N, M, P, counts, s)) != BIMASK_OK) return rc;
  return launch_pick(counts, cands, P, I, best_idx, best_perm, s);
}

int bimask_bwd_mask(const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J, int N, int M,
                    uint32_t* maskbits_b, uint16_t* vals_b, uint32_t* meta_b, void* hw_meta_b, void* stream) {
  bool pack = false;
  int rc = check_shape(I, J, N, M, &pack);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(W && maskbits_f && perm && maskbits_b, BIMASK_EINVAL, "bimask_bwd_mask: null pointer");
  if (pack) {
    BIMASK_REQUIRE(vals_b && meta_b && hw_meta_b, BIMASK_EINVAL, "bimask_bwd_mask: null pointer");
  } else {
    BIMASK_REQUIRE(!meta_b && !hw_meta_b, BIMASK_EUNSUPPORTED,
                   "N:M = %d:%d does not fit the 2:4 container: pass meta_b = hw_meta_b = NULL (vals_b, when given, receives the "
                   "dense masked operand)",
                   N, M);
  }
  BIMASK_REQUIRE(aligned16(W) && aligned16(maskbits_f) && aligned16(perm) && aligned16(maskbits_b) &&
                     aligned16(vals_b) && aligned16(meta_b) && aligned16(hw_meta_b),
                 BIMASK_EINVAL, "bimask_bwd_mask: pointers must be 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  if (M != 4) {
    const bool gfused = pack && (I % 128 == 0) && (J % 128 == 0);
    if ((rc = launch_bwd_mask_generic(W, maskbits_f, perm, I, J, N, M, maskbits_b, vals_b, meta_b, pack ? 1 : vals_b ? 2 : 0,
                                      gfused ? hw_meta_b : nullptr, s)) != BIMASK_OK)
      return rc;
    return pack && !gfused ? launch_hw_meta(meta_b, J, I, hw_meta_b, s) : BIMASK_OK;
  }
  return launch_bwd_mask(W, maskbits_f, perm, I, J, N, maskbits_b, vals_b, meta_b, hw_meta_b, s);
}

int bimask_bwd_mask_criterion(const float* W, const float* S, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                              int N, int M, int criterion, uint64_t seed, uint32_t* maskbits_b, uint16_t* vals_b,
                              uint32_t* meta_b, void* hw_meta_b, void* stream) {
  BIMASK_REQUIRE(criterion >= BIMASK_CRIT_WEIGHT && criterion <= BIMASK_CRIT_RANDOM, BIMASK_EINVAL,
                 "bimask_bwd_mask_criterion: criterion %d out of range 0..3", criterion);
  if (criterion == BIMASK_CRIT_WEIGHT)
    return bimask_bwd_mask(W, maskbits_f, perm, I, J, N, M, maskbits_b, vals_b, meta_b, hw_meta_b, stream);
  bool pack = false;
  int rc = check_shape(I, J, N, M, &pack);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(W && maskbits_f && perm && maskbits_b, BIMASK_EINVAL, "bimask_bwd_mask_criterion: null pointer");
  BIMASK_REQUIRE(criterion != BIMASK_CRIT_SCORE || S, BIMASK_EINVAL, "bimask_bwd_mask_criterion: the score criterion needs S");
  if (pack) {
    BIMASK_REQUIRE(vals_b && meta_b && hw_meta_b, BIMASK_EINVAL, "bimask_bwd_mask_criterion: null pointer");
  } else {
    BIMASK_REQUIRE(!meta_b && !hw_meta_b, BIMASK_EUNSUPPORTED,
                   "N:M = %d:%d does not fit the 2:4 container: pass meta_b = hw_meta_b = NULL (vals_b, when given, receives the "
                   "dense masked operand)",
                   N, M);
  }
  BIMASK_REQUIRE(aligned16(W) && aligned16(S) && aligned16(maskbits_f) && aligned16(perm) && aligned16(maskbits_b) &&
                     aligned16(vals_b) && aligned16(meta_b) && aligned16(hw_meta_b),
                 BIMASK_EINVAL, "bimask_bwd_mask_criterion: pointers must be 16-byte aligned");
  cudaStream_t s = (cudaStream_t)stream;
  const bool gfused = pack && (I % 128 == 0) && (J % 128 == 0);
  if ((rc = launch_bwd_mask_criterion(W, S, maskbits_f, perm, I, J, N, M, criterion, seed, maskbits_b, vals_b, meta_b,
                                      pack ? 1 : vals_b ? 2 : 0, gfused ? hw_meta_b : nullptr, s)) != BIMASK_OK)
    return rc;
  return pack && !gfused ? launch_hw_meta(meta_b, J, I, hw_meta_b, s) : BIMASK_OK;
}

static int check_gemm(int T, int I, int J) {
  BIMASK_REQUIRE(T > 0 && I > 0 && J > 0 && I % 32 == 0 && J % 32 == 0, BIMASK_EINVAL,
                 "T = %d, I = %d, J = %d: T positive, I and J positive multiples of 32", T, I, J);
  return BIMASK_OK;
}

int bimask_spmm_fwd(const uint16_t* X, const uint16_t* vals_f, const void* hw_meta_f, int T, int I, int J,
                    uint16_t* Y, int32_t* status_word, void* stream) {
  int rc = check_gemm(T, I, J);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(X && vals_f && Y && status_word, BIMASK_EINVAL, "bimask_spmm_fwd: null pointer");
  BIMASK_REQUIRE(aligned16(X) && aligned16(vals_f) && aligned16(hw_meta_f) && aligned16(Y), BIMASK_EINVAL,
                 "bimask_spmm_fwd: pointers must be 16-byte aligned");
  if (!hw_meta_f) return launch_dense_nt(vals_f, X, I, T, J, Y, status_word, (cudaStream_t)stream);
  return launch_spmm(vals_f, hw_meta_f, X, I, T, J, Y, status_word, (cudaStream_t)stream);
}

int bimask_spmm_dgrad(const uint16_t* dY, const int32_t* perm, const uint16_t* vals_b, const void* hw_meta_b,
                      int T, int I, int J, uint16_t* dX, void* ws, size_t ws_bytes, int32_t* status_word,
                      void* stream) {
  int rc = check_gemm(T, I, J);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(dY && perm && vals_b && dX && status_word && ws, BIMASK_EINVAL, "bimask_spmm_dgrad: null pointer");
  BIMASK_REQUIRE(aligned16(dY) && aligned16(perm) && aligned16(vals_b) && aligned16(hw_meta_b) && aligned16(dX) &&
                     aligned16(ws),
                 BIMASK_EINVAL, "bimask_spmm_dgrad: pointers must be 16-byte aligned");
  BIMASK_REQUIRE((size_t)I * 4 <= 200 * 1024, BIMASK_EUNSUPPORTED, "I = %d too large for the column permute pass (limit 51200)", I);
  const WsPlan w = plan_ws(T, I, J, 0);
  BIMASK_REQUIRE(ws_bytes >= w.dyp_off + w.dyp_bytes, BIMASK_EINVAL,
                 "bimask_spmm_dgrad: workspace too small (%zu bytes, need %zu)", ws_bytes, w.dyp_off + w.dyp_bytes);
  uint16_t* dYp = reinterpret_cast<uint16_t*>(reinterpret_cast<uint8_t*>(ws) + w.dyp_off);
  cudaStream_t s = (cudaStream_t)stream;
  if ((rc = launch_permute_cols(dY, perm, T, I, dYp, s)) != BIMASK_OK) return rc;
  if (!hw_meta_b) return launch_dense_nt(vals_b, dYp, J, T, I, dX, status_word, s);
  return launch_spmm(vals_b, hw_meta_b, dYp, J, T, I, dX, status_word, s);
}

int bimask_wgrad(const uint16_t* dY, const uint16_t* X, int T, int I, int J, float* dW, void* ws, size_t ws_bytes,
                 int32_t* status_word, void* stream) {
  int rc = check_gemm(T, I, J);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(dY && X && dW && status_word, BIMASK_EINVAL, "bimask_wgrad: null pointer");
  BIMASK_REQUIRE(aligned16(dY) && aligned16(X) && aligned16(dW) && (!ws || aligned16(ws)), BIMASK_EINVAL,
                 "bimask_wgrad: pointers must be 16-byte aligned");
  const WsPlan w = plan_ws(T, I, J, 0);
  float* partials = nullptr;
  if (w.part_bytes) {
    BIMASK_REQUIRE(ws && ws_bytes >= w.part_off + w.part_bytes, BIMASK_EINVAL,
                   "bimask_wgrad: workspace too small (%zu bytes, need %zu)", ws_bytes, w.part_off + w.part_bytes);
    partials = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(ws) + w.part_off);
  }
  return launch_wgrad_impl(dY, X, T, I, J, dW, partials, status_word, (cudaStream_t)stream);
}

}  // extern "C"

// A 3x3 convolution layer seen by the layer step: geometry, which products fetch shifted pixel
// patches themselves (implicit) and the column-space scratch of those that do not.
struct ConvPlan {
  int NB, H, W, C, stride;
  bool imp_fwd, imp_dgrad, imp_wgrad;
  uint16_t* xcol;     // T x 9C, when the forward or weight-gradient product is explicit
  uint16_t* dxcol;    // T x 9C, when the input gradient is explicit
  float* wpart;       // split-K partial sums of the implicit weight gradient
};

// A layer step is a chain of short kernels.  On small layers the kernels are too short to fill the GPU and the
// step takes as long as its longest dependent chain, so there the step is spread over four streams of the library's own:
//   stream H (highest priority):  forward mask -> count candidates -> backward mask -> sparse input gradient
//   stream C (highest priority):  candidate generation (needs the seed alone) ... column permutation of dY (needs the
//                                 permutation alone; the input gradient waits for it)
//   stream A (lowest priority):   dense weight gradient (needs dY and X alone)
//   stream B (lowest priority):   [metadata image of a padded forward operand ->] sparse forward product (needs the
//                                 forward mask alone)
// forked from the caller's stream after the inputs are ready and joined into it before the step returns, so the caller
// sees one ordered step.  The dependent chain has its own stream because priorities are relative to the caller's
// stream otherwise: where thread blocks of the chain and of the two independent products are waiting for an SM, the
// chain's go first (measured on the ViT block: 14.4 k -> 14.9 k layer-steps/s; the ResNet layers do not care).
// Four streams and nine events per device and host thread, created on first use and kept until exit.  (On the large
// configuration co-resident kernels contend for issue slots and the step gets slower, so there everything stays in line.)
namespace bimask {
struct SideStream {
  cudaStream_t a = nullptr, b = nullptr, c = nullptr, h = nullptr;
  cudaEvent_t fork = nullptr, gen_done = nullptr, mask_done = nullptr, perm_done = nullptr, permuted = nullptr,
              join_a = nullptr, join_b = nullptr, join_c = nullptr, join_h = nullptr;
};
static int get_side_stream(SideStream** out) {
  static thread_local SideStream side[64];
  int dev = 0;
  BIMASK_CUDA_OK(cudaGetDevice(&dev));
  BIMASK_REQUIRE(dev >= 0 && dev < 64, BIMASK_EUNSUPPORTED, "device ordinal %d out of range", dev);
  SideStream& sd = side[dev];
  if (!sd.a) {
    // the dependent chain (h) and what it waits for (c) get the highest stream priority, the two products that only
    // have to be done by the end of the step (a, b) the lowest: where thread blocks of both kinds are waiting for an SM,
    // the chain's go first
    int least = 0, greatest = 0;
    BIMASK_CUDA_OK(cudaDeviceGetStreamPriorityRange(&least, &greatest));
    BIMASK_CUDA_OK(cudaStreamCreateWithPriority(&sd.a, cudaStreamNonBlocking, least));
    BIMASK_CUDA_OK(cudaStreamCreateWithPriority(&sd.b, cudaStreamNonBlocking, least));
    BIMASK_CUDA_OK(cudaStreamCreateWithPriority(&sd.c, cudaStreamNonBlocking, greatest));
    BIMASK_CUDA_OK(cudaStreamCreateWithPriority(&sd.h, cudaStreamNonBlocking, greatest));
    for (cudaEvent_t* e : {&sd.fork, &sd.gen_done, &sd.mask_done, &sd.perm_done, &sd.permuted,
                           &sd.join_a, &sd.join_b, &sd.join_c, &sd.join_h})
      BIMASK_CUDA_OK(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
  }
  *out = &sd;
  return BIMASK_OK;
}
// Joins the side streams back into the caller's stream when the layer step leaves, on every path.
struct SideJoin {
  SideStream* side = nullptr;
  cudaStream_t main = nullptr;
  bool a_forked = false, b_forked = false, c_forked = false, h_forked = false;
  ~SideJoin() {
    if (!side) return;
    if (h_forked && cudaEventRecord(side->join_h, side->h) == cudaSuccess) cudaStreamWaitEvent(main, side->join_h, 0);
    if (a_forked && cudaEventRecord(side->join_a, side->a) == cudaSuccess) cudaStreamWaitEvent(main, side->join_a, 0);
    if (b_forked && cudaEventRecord(side->join_b, side->b) == cudaSuccess) cudaStreamWaitEvent(main, side->join_b, 0);
    if (c_forked && cudaEventRecord(side->join_c, side->c) == cudaSuccess) cudaStreamWaitEvent(main, side->join_c, 0);
  }
};
}  // namespace bimask

// skip_fwd_mask: the forward mask / operand of the current W is already in place.
// conv: null for a linear layer; otherwise a->X is x (T x C) and a->dX is dx (T x C).
static int layer_step_impl(const bimask_layer_args* a, bool skip_fwd_mask, const ConvPlan* conv = nullptr) {
  BIMASK_REQUIRE(a != nullptr, BIMASK_EINVAL, "bimask_layer_step: null argument block");
  bool pack = false;
  int rc = check_shape(a->I, a->J, a->N, a->M, &pack);
  if (rc != BIMASK_OK) return rc;
  BIMASK_REQUIRE(pack || a->N <= 4 || a->N == a->M || !a->do_search, BIMASK_EUNSUPPORTED,
                 "N:M = %d:%d: the count kernel of the search handles N <= 4", a->N, a->M);
  if ((rc = check_gemm(a->T, a->I, a->J)) != BIMASK_OK) return rc;
  BIMASK_REQUIRE(a->perm && a->ws && a->status_word && aligned16(a->ws), BIMASK_EINVAL,
                 "bimask_layer_step: null or misaligned pointer");
  BIMASK_REQUIRE(a->W && a->X && a->dY && a->Y && a->dX && a->dW && a->maskbits_f && a->vals_f && a->maskbits_b && a->vals_b,
                 BIMASK_EINVAL, "bimask_layer_step: null pointer");
  // patterns that fit the 2:4 container need the index metadata buffers; the others run the
  // products on dense masked operands (vals_f / vals_b then hold I*J bf16) and ignore them
  BIMASK_REQUIRE(!pack || (a->meta_f && a->hw_meta_f && a->meta_b && a->hw_meta_b), BIMASK_EINVAL,
                 "bimask_layer_step: null metadata pointer");
  BIMASK_REQUIRE(aligned16(a->W) && aligned16(a->X) && aligned16(a->dY) && aligned16(a->Y) && aligned16(a->dX) &&
                     aligned16(a->dW) && aligned16(a->perm) && aligned16(a->maskbits_f) && aligned16(a->vals_f) &&
                     aligned16(a->meta_f) && aligned16(a->hw_meta_f) && aligned16(a->maskbits_b) &&
                     aligned16(a->vals_b) && aligned16(a->meta_b) && aligned16(a->hw_meta_b),
                 BIMASK_EINVAL, "bimask_layer_step: pointers must be 16-byte aligned");
  BIMASK_REQUIRE((size_t)a->I * 4 <= 200 * 1024, BIMASK_EUNSUPPORTED,
                 "I = %d too large for the column permute pass (limit 51200)", a->I);
  if (a->do_search) {
    BIMASK_REQUIRE(a->P >= 1 && a->P <= 65535 && a->best_idx && a->counts, BIMASK_EINVAL,
                   "bimask_layer_step: search needs 1 <= P <= 65535, best_idx and counts");
    BIMASK_REQUIRE(a->cands || a->I < (1 << 24), BIMASK_EUNSUPPORTED, "generated candidates need I < 2^24 (I = %d)", a->I);
  }
  // three disjoint scratch regions: generated candidates, permuted dY, split-K partials
  const WsPlan w = plan_ws(a->T, a->I, a->J, a->do_search && !a->cands ? a->P : 0);
  BIMASK_REQUIRE(a->ws_bytes >= w.total, BIMASK_EINVAL, "bimask_layer_step: workspace too small (%zu bytes, need %zu)",
                 a->ws_bytes, w.total);
  uint8_t* ws = reinterpret_cast<uint8_t*>(a->ws);
  int32_t* gen = reinterpret_cast<int32_t*>(ws + w.cands_off);
  uint16_t* dYp = reinterpret_cast<uint16_t*>(ws + w.dyp_off);
  float* partials = w.part_bytes ? reinterpret_cast<float*>(ws + w.part_off) : nullptr;

  // Alg. 1 in order on the caller's stream; small layers spread it over side streams as well (see SideStream).
  cudaStream_t s = (cudaStream_t)a->stream;
  const uint16_t* Xmat = a->X;                       // the T x J activation matrix of the explicit products
  uint16_t* dXmat = a->dX;
  if (conv) {
    Xmat = conv->xcol;
    dXmat = conv->dxcol;
    if (!conv->imp_fwd || !conv->imp_wgrad)
      if ((rc = launch_im2col3x3(a->X, conv->NB, conv->H, conv->W, conv->C, conv->stride, conv->xcol, s))) return rc;
  }
  // small layers (between a gigaflop and a hundred): side streams, see SideStream
  const double flops = 2.0 * a->T * a->I * a->J;
  const bool spread = flops >= 1e9 && flops < 1e11;
  SideJoin join;
  SideStream* side = nullptr;
  cudaStream_t sm = s;                                  // the dependent chain: masks, count, input gradient
  cudaStream_t sa = s, sb = s, sc = s;                  // weight gradient / forward product / generation + permutation of dY
  const bool gen_here = a->do_search && !a->cands;
  if (spread) {
    if ((rc = get_side_stream(&side))) return rc;
    join.side = side;
    join.main = s;
    sm = side->h;
    sa = side->a;
    sb = side->b;
    sc = side->c;
    BIMASK_CUDA_OK(cudaEventRecord(side->fork, s));
    BIMASK_CUDA_OK(cudaStreamWaitEvent(sm, side->fork, 0));
    join.h_forked = true;
    BIMASK_CUDA_OK(cudaStreamWaitEvent(sc, side->fork, 0));
    join.c_forked = true;
    BIMASK_CUDA_OK(cudaStreamWaitEvent(sa, side->fork, 0));
    join.a_forked = true;
  }
  // the 2:4 mask kernels (M = 4) write the metadata images themselves, padding included; the generic ones (M = 8, 16)
  // do so on unpadded shapes and need the re-ordering pass otherwise
  const bool fused = pack && (a->M == 4 || ((a->I % 128 == 0) && (a->J % 128 == 0)));
  if (!skip_fwd_mask) {
    if (a->M == 4)
      rc = launch_fwd_mask(a->W, a->I, a->J, a->N, a->maskbits_f, a->vals_f, a->meta_f, fused ? a->hw_meta_f : nullptr, sm);
    else
      rc = launch_fwd_mask_generic(a->W, a->I, a->J, a->N, a->M, a->maskbits_f, a->vals_f, a->meta_f, pack ? 1 : 2,
                                   fused ? a->hw_meta_f : nullptr, sm);
    if (rc) return rc;
  }
  if (spread) {
    BIMASK_CUDA_OK(cudaEventRecord(side->mask_done, sm));
    BIMASK_CUDA_OK(cudaStreamWaitEvent(sb, side->mask_done, 0));
    join.b_forked = true;
    if (gen_here) {                                      // beside the forward mask; the count kernel waits for both
      if ((rc = launch_gen_candidates(a->seed, a->P, a->I, gen, sc, a->M == 4 ? a->counts : nullptr,
                                      a->M == 4 ? a->best_idx : nullptr)))
        return rc;
      BIMASK_CUDA_OK(cudaEventRecord(side->gen_done, sc));
    }
    if (conv && conv->imp_wgrad)
      rc = launch_wgrad_conv(a->dY, a->X, conv->NB, conv->H, conv->W, conv->C, a->I, conv->stride, a->dW, conv->wpart,
                             a->status_word, sa);
    else
      rc = launch_wgrad_impl(a->dY, Xmat, a->T, a->I, a->J, a->dW, partials, a->status_word, sa);
    if (rc) return rc;
  }
  // padded shapes: the metadata image of the forward operand is a pass of its own, needed by the forward product only
  if (!skip_fwd_mask && pack && !fused && (rc = launch_hw_meta(a->meta_f, a->I, a->J, a->hw_meta_f, sb))) return rc;
  if (conv && conv->imp_fwd)
    rc = launch_spmm_conv(1, a->vals_f, a->hw_meta_f, a->X, conv->NB, conv->H, conv->W, conv->C, a->I, conv->stride, a->Y,
                          a->status_word, sb);
  else if (pack) rc = launch_spmm(a->vals_f, a->hw_meta_f, Xmat, a->I, a->T, a->J, a->Y, a->status_word, sb);
  else rc = launch_dense_nt(a->vals_f, Xmat, a->I, a->T, a->J, a->Y, a->status_word, sb);
  if (rc) return rc;
  if (a->do_search) {
    const int32_t* cands = a->cands;
    if (!cands) {
      if (spread) {
        BIMASK_CUDA_OK(cudaStreamWaitEvent(sm, side->gen_done, 0));
      } else if ((rc = launch_gen_candidates(a->seed, a->P, a->I, gen, sm, a->M == 4 ? a->counts : nullptr,
                                             a->M == 4 ? a->best_idx : nullptr))) {
        return rc;
      }
      cands = gen;
    }
    if (a->M == 4) {
      // the count kernel's last CTA picks the winner and copies it into perm
      if ((rc = launch_score(a->maskbits_f, cands, a->I, a->J, a->N, a->P, a->counts, sm, a->cands == nullptr, a->best_idx, a->perm)))
        return rc;
    } else {
      if ((rc = launch_score_generic(a->maskbits_f, cands, a->I, a->J, a->N, a->M, a->P, a->counts, sm))) return rc;
      if ((rc = launch_pick(a->counts, cands, a->P, a->I, a->best_idx, a->perm, sm))) return rc;
    }
  }
  if (spread) {                                          // the permutation is final: dY[:, perm] goes to side stream C
    BIMASK_CUDA_OK(cudaEventRecord(side->perm_done, sm));
    BIMASK_CUDA_OK(cudaStreamWaitEvent(sc, side->perm_done, 0));
    if ((rc = launch_permute_cols(a->dY, a->perm, a->T, a->I, dYp, sc))) return rc;
    BIMASK_CUDA_OK(cudaEventRecord(side->permuted, sc));
  }
  if (a->M == 4)
    rc = launch_bwd_mask(a->W, a->maskbits_f, a->perm, a->I, a->J, a->N, a->maskbits_b, a->vals_b, a->meta_b,
                         fused ? a->hw_meta_b : nullptr, sm);
  else
    rc = launch_bwd_mask_generic(a->W, a->maskbits_f, a->perm, a->I, a->J, a->N, a->M, a->maskbits_b, a->vals_b, a->meta_b,
                                 pack ? 1 : 2, fused ? a->hw_meta_b : nullptr, sm);
  if (rc) return rc;
  if (pack && !fused && (rc = launch_hw_meta(a->meta_b, a->J, a->I, a->hw_meta_b, sm))) return rc;
  if (spread) {
    BIMASK_CUDA_OK(cudaStreamWaitEvent(sm, side->permuted, 0));
  } else if ((rc = launch_permute_cols(a->dY, a->perm, a->T, a->I, dYp, sm))) {
    return rc;
  }
  if (conv && conv->imp_dgrad)
    rc = launch_spmm_conv(2, a->vals_b, a->hw_meta_b, dYp, conv->NB, conv->H, conv->W, conv->C, a->I, conv->stride, a->dX, a->status_word, sm);
  else if (pack) rc = launch_spmm(a->vals_b, a->hw_meta_b, dYp, a->J, a->T, a->I, dXmat, a->status_word, sm);
  else rc = launch_dense_nt(a->vals_b, dYp, a->J, a->T, a->I, dXmat, a->status_word, sm);
  if (rc) return rc;
  if (conv && !conv->imp_dgrad)
    if ((rc = launch_col2im3x3(dXmat, conv->NB, conv->H, conv->W, conv->C, conv->stride, a->dX, sm))) return rc;
  if (spread) return BIMASK_OK;                           // already running beside the chain; joined on return
  if (conv && conv->imp_wgrad)
    return launch_wgrad_conv(a->dY, a->X, conv->NB, conv->H, conv->W, conv->C, a->I, conv->stride, a->dW, conv->wpart,
                             a->status_word, s);
  return launch_wgrad_impl(a->dY, Xmat, a->T, a->I, a->J, a->dW, partials, a->status_word, s);
}

extern "C" {

int bimask_layer_step(const bimask_layer_args* a) { return layer_step_impl(a, false); }

static size_t conv_wpart_bytes(int NB, int H, int W, int C, int I, int stride) {
  int splits = 1, per = 0;
  wgrad_conv_plan(NB, H, W, C, I, stride, &splits, &per);
  return splits > 1 ? align_up((size_t)splits * I * 9 * C * sizeof(float), 256) : 0;
}

size_t bimask_conv_workspace_bytes(int NB, int H, int W, int C, int I, int P, int stride) {
  if (NB <= 0 || H <= 0 || W <= 0 || C <= 0 || I <= 0 || (stride != 1 && stride != 2)) return 0;
  const long long T = (long long)NB * ((H - 1) / stride + 1) * ((W - 1) / stride + 1);     // output pixels
  if (T > 0x7FFFFFFFll || 9ll * C > 0x7FFFFFFFll) return 0;
  const size_t col = align_up((size_t)T * 9 * C * 2, 256);
  // linear-layer scratch + column matrix + column-space gradient + partial sums of the implicit weight gradient
  return plan_ws((int)T, I, 9 * C, P).total + 2 * col + conv_wpart_bytes(NB, H, W, C, I, stride);
}

int bimask_conv_layer_step(const bimask_conv_args* c) {
  BIMASK_REQUIRE(c != nullptr, BIMASK_EINVAL, "bimask_conv_layer_step: null argument block");
  const bimask_layer_args* a = &c->layer;
  BIMASK_REQUIRE(c->NB > 0 && c->H > 0 && c->W > 0 && c->C > 0 && c->C % 32 == 0, BIMASK_EINVAL,
                 "bimask_conv_layer_step: NB = %d, H = %d, W = %d, C = %d: all positive, C a multiple of 32", c->NB, c->H,
                 c->W, c->C);
  BIMASK_REQUIRE(c->stride == 1 || c->stride == 2, BIMASK_EUNSUPPORTED, "bimask_conv_layer_step: stride %d (1 and 2 are implemented)",
                 c->stride);
  const long long T = (long long)c->NB * ((c->H - 1) / c->stride + 1) * ((c->W - 1) / c->stride + 1);
  BIMASK_REQUIRE(T <= 0x7FFFFFFFll && a->T == (int)T && a->J == 9 * c->C, BIMASK_EINVAL,
                 "bimask_conv_layer_step: layer.T must be the number of output pixels (%lld) and layer.J must be 9*C (%d)", T,
                 9 * c->C);
  BIMASK_REQUIRE(c->mode >= BIMASK_CONV_AUTO && c->mode <= BIMASK_CONV_IMPLICIT, BIMASK_EINVAL,
                 "bimask_conv_layer_step: mode %d out of range", c->mode);
  BIMASK_REQUIRE(a->ws && aligned16(a->ws), BIMASK_EINVAL, "bimask_conv_layer_step: null or misaligned workspace");
  const size_t need = bimask_conv_workspace_bytes(c->NB, c->H, c->W, c->C, a->I, a->do_search && !a->cands ? a->P : 0, c->stride);
  BIMASK_REQUIRE(a->ws_bytes >= need, BIMASK_EINVAL, "bimask_conv_layer_step: workspace too small (%zu bytes, need %zu)",
                 a->ws_bytes, need);
  ConvPlan plan;
  plan.NB = c->NB; plan.H = c->H; plan.W = c->W; plan.C = c->C; plan.stride = c->stride;
  // all three products have an implicit form for both strides: the forward product and the weight gradient through a
  // strided tensor-map traversal, the input gradient of a stride-2 layer as four stride-1 problems, one per parity
  // class of the input pixels.  The input gradient needs whole 128-row operand tiles per filter tap (C % 128 == 0, or
  // C = 64); where it cannot go implicit (other C % 64 == 0) it keeps the explicit form beside the implicit others.
  const bool packs = a->N <= 2;
  const bool can_fwd = packs && c->C % 64 == 0;
  const bool can_dgrad = packs && (c->C % 128 == 0 || c->C == 64);
  const bool can_wgrad = c->C % 64 == 0;
  BIMASK_REQUIRE(c->mode != BIMASK_CONV_IMPLICIT || (can_fwd && can_wgrad), BIMASK_EUNSUPPORTED,
                 "bimask_conv_layer_step: the implicit form needs C %% 64 == 0 and a pattern with a 2:4 form "
                 "(stride %d, C = %d, I = %d, N:M = %d:%d)", c->stride, c->C, a->I, a->N, a->M);
  // AUTO: a column matrix that fits comfortably in L2 costs little, and the explicit form then has
  // fewer, denser k tiles (measured: 7x7 images of 512 channels are faster explicit, 14x14 of 256
  // channels faster implicit); above 16 MiB the implicit form wins by the HBM traffic it avoids.
  // Images of at most 8 x 8 output pixels leave a quarter of every pixel box empty, more than the unfold and fold
  // passes cost (measured at batch 256, 7x7 x 512 channels: 256 us explicit, 295 us implicit).
  const bool small_cols = (size_t)T * 9 * c->C * 2 < ((size_t)16 << 20);
  const bool small_image = T / c->NB <= 64;
  const bool implicit = c->mode == BIMASK_CONV_IMPLICIT || (c->mode == BIMASK_CONV_AUTO && !small_cols && !small_image);
  plan.imp_fwd = implicit && can_fwd;
  plan.imp_dgrad = implicit && can_dgrad;
  plan.imp_wgrad = implicit && can_wgrad;
  const size_t col = align_up((size_t)T * 9 * c->C * 2, 256);
  const size_t wpart = conv_wpart_bytes(c->NB, c->H, c->W, c->C, a->I, c->stride);
  uint8_t* tail = reinterpret_cast<uint8_t*>(a->ws) + (need - 2 * col - wpart);
  plan.xcol = reinterpret_cast<uint16_t*>(tail);
  plan.dxcol = reinterpret_cast<uint16_t*>(tail + col);
  plan.wpart = reinterpret_cast<float*>(tail + 2 * col);
  return layer_step_impl(a, false, &plan);
}

int bimask_train_step(const bimask_train_args* a) {
  BIMASK_REQUIRE(a != nullptr, BIMASK_EINVAL, "bimask_train_step: null argument block");
  BIMASK_REQUIRE(a->t >= 1 && a->delta_t >= 1, BIMASK_EINVAL, "bimask_train_step: t = %lld and delta_t = %d must be >= 1",
                 (long long)a->t, a->delta_t);
  BIMASK_REQUIRE(a->lr == a->lr && a->momentum == a->momentum && a->weight_decay == a->weight_decay, BIMASK_EINVAL,
                 "bimask_train_step: NaN hyper-parameter");
  BIMASK_REQUIRE(aligned16(a->mom), BIMASK_EINVAL, "bimask_train_step: mom must be 16-byte aligned");
  bimask_layer_args l = a->layer;
  l.do_search = (a->t % a->delta_t == 0) ? 1 : 0;
  l.seed = a->layer.seed + (uint64_t)(a->t / a->delta_t);       // a fresh draw per interval
  int rc = layer_step_impl(&l, a->premasked != 0);
  if (rc != BIMASK_OK) return rc;
  // the update reads dW after the weight-gradient kernel on the same stream, then the next mask
  const bool pack = l.N <= 2;      // otherwise vals_f is the dense masked operand and there is no metadata
  return bimask_sgd_fwd_mask(const_cast<float*>(l.W), l.dW, a->mom, l.I, l.J, l.N, l.M, a->lr, a->momentum,
                             a->weight_decay, l.maskbits_f, l.vals_f, pack ? l.meta_f : nullptr,
                             pack ? l.hw_meta_f : nullptr, l.stream);
}

}  // extern "C"

namespace bimask {

// Copy streams and events of the host-buffer entry points, one set per device, created on first
// use and kept until exit.  The last four calls are remembered (which device buffers they read and
// wrote, and their three events) so that a new call waits only for earlier calls it shares buffers
// with: a caller that alternates between buffer sets gets uploads, kernels and downloads of
// different calls running at the same time.
struct HostSlot {
  const void* in[4];                 // device buffers the upload writes: W, X, dY, perm
  const void* out[12];               // device buffers the kernels write / the download reads
  cudaEvent_t in_done = nullptr, compute_done = nullptr, out_done = nullptr;
  cudaStream_t stream = nullptr;
  bool used = false;
};
struct HostPipe {
  cudaStream_t in = nullptr, out = nullptr;
  HostSlot slots[4];
  int next = 0;
  bool ready = false, used = false;
};
static std::mutex g_pipe_mutex;
static HostPipe g_pipes[64];

static int get_pipe(HostPipe** out) {
  int dev = 0;
  BIMASK_CUDA_OK(cudaGetDevice(&dev));
  BIMASK_REQUIRE(dev >= 0 && dev < 64, BIMASK_EUNSUPPORTED, "device ordinal %d out of range", dev);
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  HostPipe& p = g_pipes[dev];
  if (!p.ready) {
    BIMASK_CUDA_OK(cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking));
    BIMASK_CUDA_OK(cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking));
    for (HostSlot& sl : p.slots) {
      BIMASK_CUDA_OK(cudaEventCreateWithFlags(&sl.in_done, cudaEventDisableTiming));
      BIMASK_CUDA_OK(cudaEventCreateWithFlags(&sl.compute_done, cudaEventDisableTiming));
      BIMASK_CUDA_OK(cudaEventCreateWithFlags(&sl.out_done, cudaEventDisableTiming));
    }
    p.ready = true;
  }
  *out = &p;
  return BIMASK_OK;
}

static bool shares(const void* const* a, int na, const void* const* b, int nb) {
  for (int i = 0; i < na; ++i)
    for (int k = 0; k < nb; ++k)
      if (a[i] != nullptr && a[i] == b[k]) return true;
  return false;
}

}  // namespace bimask

extern "C" {

int bimask_layer_step_host_async(const bimask_layer_args* d, const bimask_layer_args* h, int32_t* host_status_word) {
  BIMASK_REQUIRE(d && h, BIMASK_EINVAL, "bimask_layer_step_host: null argument block");
  BIMASK_REQUIRE(h->W && h->X && h->dY, BIMASK_EINVAL, "bimask_layer_step_host: host W, X and dY are required");
  BIMASK_REQUIRE(d->W && d->X && d->dY && d->status_word, BIMASK_EINVAL, "bimask_layer_step_host: null device pointer");
  HostPipe* p = nullptr;
  int rc = get_pipe(&p);
  if (rc != BIMASK_OK) return rc;
  cudaStream_t s = (cudaStream_t)d->stream;
  const size_t IJ = (size_t)d->I * d->J, TJ = (size_t)d->T * d->J, TI = (size_t)d->T * d->I;
  // Three queues: inputs go up on `in`, the step runs on the caller's stream, results come down
  // on `out` (PCIe is full duplex).  An upload waits for the kernels of earlier calls that used the
  // device buffers it overwrites; the kernels wait for their own upload and for the downloads of
  // earlier calls that read the buffers they overwrite.
  HostSlot* me = &p->slots[p->next];
  const void* ins[4] = {d->W, d->X, d->dY, d->perm};
  const void* outs[12] = {d->Y, d->dX, d->dW, d->perm, d->counts, d->best_idx, d->maskbits_f, d->maskbits_b,
                          d->status_word, d->vals_f, d->vals_b, d->ws};
  if (!p->used) {
    // order behind whatever the caller's stream already holds
    BIMASK_CUDA_OK(cudaEventRecord(me->compute_done, s));
    BIMASK_CUDA_OK(cudaStreamWaitEvent(p->in, me->compute_done, 0));
  }
  for (HostSlot& o : p->slots) {
    if (!o.used) continue;
    const bool evicted = &o == me;                       // its record is about to be overwritten: depend on it
    const bool in_hit = evicted || shares(ins, 4, o.in, 4) || shares(ins, 4, o.out, 12);
    const bool out_hit = evicted || shares(outs, 12, o.out, 12) || shares(outs, 12, o.in, 4);
    if (in_hit) BIMASK_CUDA_OK(cudaStreamWaitEvent(p->in, o.compute_done, 0));
    if (in_hit && shares(ins, 4, o.out, 12)) BIMASK_CUDA_OK(cudaStreamWaitEvent(p->in, o.out_done, 0));
    if (out_hit) BIMASK_CUDA_OK(cudaStreamWaitEvent(s, o.out_done, 0));
    if ((in_hit || out_hit) && o.stream != s) BIMASK_CUDA_OK(cudaStreamWaitEvent(s, o.compute_done, 0));
  }
  BIMASK_CUDA_OK(cudaMemcpyAsync(const_cast<float*>(d->W), h->W, IJ * 4, cudaMemcpyHostToDevice, p->in));
  BIMASK_CUDA_OK(cudaMemcpyAsync(const_cast<uint16_t*>(d->X), h->X, TJ * 2, cudaMemcpyHostToDevice, p->in));
  BIMASK_CUDA_OK(cudaMemcpyAsync(const_cast<uint16_t*>(d->dY), h->dY, TI * 2, cudaMemcpyHostToDevice, p->in));
  if (!d->do_search && h->perm)
    BIMASK_CUDA_OK(cudaMemcpyAsync(d->perm, h->perm, (size_t)d->I * 4, cudaMemcpyHostToDevice, p->in));
  if (d->do_search && d->cands && h->cands)
    BIMASK_CUDA_OK(cudaMemcpyAsync(const_cast<int32_t*>(d->cands), h->cands, (size_t)d->P * d->I * 4,
                                   cudaMemcpyHostToDevice, p->in));
  BIMASK_CUDA_OK(cudaEventRecord(me->in_done, p->in));
  BIMASK_CUDA_OK(cudaStreamWaitEvent(s, me->in_done, 0));
  BIMASK_CUDA_OK(cudaMemsetAsync(d->status_word, 0, sizeof(int32_t), s));
  rc = bimask_layer_step(d);
  // even when the step refused to launch, leave the queues in a consistent state
  BIMASK_CUDA_OK(cudaEventRecord(me->compute_done, s));
  for (int i = 0; i < 4; ++i) me->in[i] = ins[i];
  for (int i = 0; i < 12; ++i) me->out[i] = outs[i];
  me->stream = s;
  me->used = true;
  p->used = true;
  p->next = (p->next + 1) % 4;
  if (rc != BIMASK_OK) {
    BIMASK_CUDA_OK(cudaEventRecord(me->out_done, s));
    return rc;
  }
  BIMASK_CUDA_OK(cudaStreamWaitEvent(p->out, me->compute_done, 0));
  cudaStream_t o = p->out;
  if (h->Y) BIMASK_CUDA_OK(cudaMemcpyAsync(h->Y, d->Y, TI * 2, cudaMemcpyDeviceToHost, o));
  if (h->dX) BIMASK_CUDA_OK(cudaMemcpyAsync(h->dX, d->dX, TJ * 2, cudaMemcpyDeviceToHost, o));
  if (h->dW) BIMASK_CUDA_OK(cudaMemcpyAsync(h->dW, d->dW, IJ * 4, cudaMemcpyDeviceToHost, o));
  if (h->perm) BIMASK_CUDA_OK(cudaMemcpyAsync(h->perm, d->perm, (size_t)d->I * 4, cudaMemcpyDeviceToHost, o));
  if (d->do_search && h->best_idx) BIMASK_CUDA_OK(cudaMemcpyAsync(h->best_idx, d->best_idx, 4, cudaMemcpyDeviceToHost, o));
  if (d->do_search && h->counts)
    BIMASK_CUDA_OK(cudaMemcpyAsync(h->counts, d->counts, (size_t)d->P * 8, cudaMemcpyDeviceToHost, o));
  if (h->maskbits_f) BIMASK_CUDA_OK(cudaMemcpyAsync(h->maskbits_f, d->maskbits_f, IJ / 8, cudaMemcpyDeviceToHost, o));
  if (h->maskbits_b) BIMASK_CUDA_OK(cudaMemcpyAsync(h->maskbits_b, d->maskbits_b, IJ / 8, cudaMemcpyDeviceToHost, o));
  if (host_status_word) BIMASK_CUDA_OK(cudaMemcpyAsync(host_status_word, d->status_word, 4, cudaMemcpyDeviceToHost, o));
  BIMASK_CUDA_OK(cudaEventRecord(me->out_done, o));
  return BIMASK_OK;
}

// Waits until every download enqueued so far on this device is in host memory.
int bimask_host_sync(void) {
  HostPipe* p = nullptr;
  int rc = get_pipe(&p);
  if (rc != BIMASK_OK) return rc;
  if (p->used) BIMASK_CUDA_OK(cudaStreamSynchronize(p->out));
  return BIMASK_OK;
}

int bimask_layer_step_host(const bimask_layer_args* d, const bimask_layer_args* h, int32_t* host_status_word) {
  int rc = bimask_layer_step_host_async(d, h, host_status_word);
  if (rc != BIMASK_OK) return rc;
  return bimask_host_sync();
}

int bimask_debug_wait_probe(int32_t* status_word, void* stream) {
  BIMASK_REQUIRE(status_word != nullptr, BIMASK_EINVAL, "bimask_debug_wait_probe: null pointer");
  return launch_wait_probe(status_word, (cudaStream_t)stream);
}

int bimask_debug_status(int32_t* out) {
  BIMASK_REQUIRE(out != nullptr, BIMASK_EINVAL, "bimask_debug_status: null pointer");
  out[0] = out[1] = out[2] = out[3] = 0;
#ifndef BIMASK_DEBUG
  set_error("bimask_debug_status: this library was built without BIMASK_DEBUG");
  return BIMASK_EUNSUPPORTED;
#else
  int (*collect[4])(int*) = {debug_collect_mask, debug_collect_perm, debug_collect_gemm_host, debug_collect_generic};
  for (auto fn : collect) {
    int rec[4];
    const int rc = fn(rec);
    if (rc != BIMASK_OK) return rc;
    if (rec[0] != 0 && out[0] == 0) { out[0] = rec[0]; out[1] = rec[1]; out[2] = rec[2]; out[3] = rec[3]; }
  }
  return BIMASK_OK;
#endif
}

int bimask_debug_gen_candidates(uint64_t seed, int P, int I, int part_cap, int32_t* cands, void* stream) {
  BIMASK_REQUIRE(cands != nullptr && aligned16(cands), BIMASK_EINVAL, "bimask_debug_gen_candidates: null or misaligned pointer");
  BIMASK_REQUIRE(P >= 1 && P <= 65535 && I >= 1 && I < (1 << 24) && part_cap >= 0, BIMASK_EINVAL,
                 "bimask_debug_gen_candidates: P = %d, I = %d, part_cap = %d out of range", P, I, part_cap);
  return launch_gen_candidates(seed, P, I, cands, (cudaStream_t)stream, nullptr, nullptr, part_cap);
}

int bimask_check_perms(const int32_t* cands, int P, int I, int32_t* ok, void* ws, size_t ws_bytes, void* stream) {
  BIMASK_REQUIRE(cands && ok && ws && P >= 1 && I >= 1, BIMASK_EINVAL, "bimask_check_perms: bad argument");
  BIMASK_REQUIRE(ws_bytes >= (size_t)P * I, BIMASK_EINVAL, "bimask_check_perms: workspace too small");
  return launch_check_perms(cands, P, I, ok, reinterpret_cast<uint8_t*>(ws), (cudaStream_t)stream);
}

}  // extern "C"
