/*
 * bimask.h -- C ABI of the Bi-Mask per-layer sparse training step on one B200 (sm_100a).
 *
 * The step follows "Bi-directional Masks for Efficient N:M Sparse Training" (Alg. 1):
 * forward N:M mask (Eq. 4), sparse forward product (Eq. 3), row-permutation search
 * (the permutation step of Alg. 1: the candidate with the most eligible blocks wins), backward mask on the
 * permuted weights (Eq. 11), sparse input-gradient product (Eq. 10) and the dense
 * straight-through weight gradient (Sec. 3.1).
 *
 * Conventions for every call unless stated otherwise
 *   - All matrices are row-major and dense.  W is I x J fp32 (output rows x input dim),
 *     X is T x J bf16, dY is T x I bf16 (bf16 is passed as uint16_t bit patterns).
 *   - Every pointer is a DEVICE pointer owned by the caller, 16-byte aligned.  The library
 *     allocates nothing, frees nothing and never synchronises: work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream).  Kernels are launched
 *     with programmatic stream serialization and wait for the work before them on the stream
 *     before they touch global memory: relative to other work of the caller on the same
 *     stream they behave like ordinary launches, and every call may be captured in a CUDA graph.
 *   - Outputs are fully overwritten, inputs are never modified.
 *   - Return value: BIMASK_OK or a negative bimask_status.  On a negative return caused by
 *     argument validation nothing was launched.  bimask_last_error() gives a text for the
 *     calling thread's last failure.
 *   - Shapes: I % 32 == 0, J % 32 == 0.  Patterns: M in {4, 8, 16}.  With N <= 2 (2:4, 1:4, 2:8,
 *     1:8, 1:16, ...) every aligned group of four holds at most two survivors, so the result is
 *     packed into the 2:4 container (a spare slot holds +0) and the products run on the sparse
 *     tensor cores.  With N > 2 (4:8, the one such pattern in the paper) no hardware format
 *     exists: there is no index metadata (meta and hw_meta must be NULL in the mask calls), and
 *     `vals`, when given, receives the DENSE masked operand instead -- I*J bf16, kept weights
 *     rounded to bf16 and +0 elsewhere, row-major like the matrix it stands for (vals_f: I x J,
 *     vals_b: J x I in permuted row order).  bimask_spmm_fwd / bimask_spmm_dgrad called with
 *     hw_meta == NULL take that dense operand and run a dense tensor-core product;
 *     bimask_layer_step / bimask_train_step do the same by themselves (their meta / hw_meta
 *     fields are then ignored and vals_f / vals_b must hold I*J bf16).  M = 4 with N > 2 is not
 *     implemented; the search counts eligible blocks for N <= 4 or N == M.
 *   - `perm[k]` is the source row of permuted row k (gather: Wp[k,:] = W[perm[k],:]), 0-based.
 *   - Device-side trouble (a bounded wait that ran out) is reported by writing a non-zero
 *     code into *status_word (a device int the caller reads when it chooses to sync);
 *     kernels never trap.
 *
 * Packed 2:4 operand ("vals" + "meta", not defined by the paper; it is the tensor core's
 * compressed format written row by row):
 *   per aligned group g of 4 consecutive elements of a row: S = kept positions ascending.
 *   |S| = 2: (idx0, idx1) = S.  |S| < 2: pad with the lowest positions not in S, sort.
 *   vals[row][2g + s] = bf16_rne(value at idx_s) if idx_s in S else +0.
 *   code = idx0 | idx1 << 2, stored in bits [4 (g % 8), +4) of meta[row][g / 8].
 *   maskbits[row][c / 32] bit (c % 32) = mask at column c.
 *   "hw_meta" is an opaque re-ordering of meta for the tensor core; size from
 *   bimask_hw_meta_bytes(rows, K).
 */
#ifndef BIMASK_H
#define BIMASK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BIMASK_OK = 0,
  BIMASK_EINVAL = -1,       /* null / misaligned pointer, bad shape, N or P out of range, workspace too small */
  BIMASK_EUNSUPPORTED = -2, /* pattern or block length not implemented, metadata asked for a pattern without a 2:4 form, size beyond a kernel limit */
  BIMASK_ECUDA = -3,        /* a CUDA call failed; see bimask_last_error() */
  BIMASK_ETIMEOUT = -4,     /* value written to *status_word when a device-side bounded wait ran out */
  BIMASK_EBOUNDS = -5       /* debug build only: a caller-supplied row index (perm / candidate entry) was out of range */
} bimask_status;

/* Text of the calling thread's last error ("" if none).  Host memory owned by the library. */
const char* bimask_last_error(void);

/* Number of kernels this library has launched in this process so far (all threads). */
uint64_t bimask_launch_count(void);

/* Bytes of the opaque tensor-core metadata buffer for a packed operand with `rows` rows and
 * reduction length K (K = J for the forward operand, K = I for the backward one). */
size_t bimask_hw_meta_bytes(int rows, int K);

/* Bytes of scratch (`ws`) large enough for every call below on a layer of this size. */
size_t bimask_workspace_bytes(int T, int I, int J, int P);

/* Eq. 4 + packing.  Forward mask: in every row, every aligned block of M along J keeps its N
 * largest |W| (ties: lowest index), compared on the fp32 values.
 *   W          in   I x J fp32
 *   maskbits_f out  I x J/32 u32
 *   vals_f     out  I x J/2 bf16,  meta_f out I x J/32 u32,  hw_meta_f out (opaque) */
int bimask_fwd_mask(const float* W, int I, int J, int N, int M,
                    uint32_t* maskbits_f, uint16_t* vals_f, uint32_t* meta_f, void* hw_meta_f,
                    void* stream);

/* Alg. 1, permutation step.  counts[c] = number of (row block k, column l) whose M rows
 * cand_c[kM .. kM+M-1] hold at most N forward-mask bits in column l ("eligible N:M blocks");
 * best_idx = lowest c with the largest count; best_perm = cand_best.
 *   cands_or_null  in   P x I i32 explicit candidates (each a permutation of 0..I-1), or NULL:
 *                       then candidate c is generated from `seed` by sorting the rows by the
 *                       key  mix64(mix64(seed + 0x9E3779B97F4A7C15 (c+1)) ^ i)  (low 24 bits
 *                       replaced by i; mix64 = SplitMix64's output function).  Needs I < 2^24.
 *   This call alone accepts any I % M == 0 (the packed operands need I % 32 == 0); for M = 8, 16
 *   the count kernel handles N <= 4 (and the trivial N == M).
 *   Limits: 1 <= P <= 65535 (BIMASK_EINVAL otherwise); generated candidates need I < 2^24
 *   (BIMASK_EUNSUPPORTED otherwise; explicit candidates have no such limit).
 *   best_perm out I i32, best_idx out 1 i32, counts out P i64
 *   ws: scratch of at least bimask_workspace_bytes(...) bytes (holds the generated candidates). */
int bimask_perm_search(const uint32_t* maskbits_f, int I, int J, int N, int M, int P, uint64_t seed,
                       const int32_t* cands_or_null,
                       int32_t* best_perm, int32_t* best_idx, int64_t* counts,
                       void* ws, size_t ws_bytes, void* stream);

/* Eq. 11 + transposed packing.  Backward mask on the permuted rows: in every column l, every
 * aligned block of M permuted rows keeps, among the entries with forward bit 1, the N largest
 * |W| (ties: lowest permuted row).  B-bar is a subset of B[perm].
 *   maskbits_b out I x J/32 u32, row k = B-bar of W row perm[k]
 *   vals_b out J x I/2 bf16, meta_b out J x I/32 u32: the operand (B-bar * W[perm,:])^T, 2:4
 *   along the permuted row index (the reduction dim of Eq. 10); hw_meta_b opaque. */
int bimask_bwd_mask(const float* W, const uint32_t* maskbits_f, const int32_t* perm,
                    int I, int J, int N, int M,
                    uint32_t* maskbits_b, uint16_t* vals_b, uint32_t* meta_b, void* hw_meta_b,
                    void* stream);

/* Greedy refinement of a permutation by pairwise swaps -- beyond the paper, whose conclusion names a
 * better search than "the best of K random candidates" as future work; not part of Algorithm 1.
 * Hill climbing on the quantity the search maximises (the eligible-block count): every round pairs
 * the positions of the permutation at random (pair i = (order[2i], order[2i+1]) with order the r-th
 * permutation drawn from seed + 0x5EED5EED by the candidate generator), evaluates for each pair whose
 * positions lie in different row blocks the change of the count if the two rows changed places
 * (against the permutation at the start of the round), and accepts a pair when its gain is positive
 * and it is, for BOTH of its blocks, the best pair touching that block (largest gain, lowest pair
 * index on equal gain).  Accepted pairs never share a block, so the count never decreases and the
 * result does not depend on the order of evaluation.  Typical use: bimask_perm_search, then this on
 * best_perm, then bimask_bwd_mask.  On i.i.d. weights the best of 128 random candidates sits within a
 * few 0.1 % of the mean (11/16 of the blocks at 2:4); 32 rounds add 1-4 % depending on J.
 *   perm_inout  in/out  device int32[I], a permutation of 0..I-1
 *   count_out   out     device int64, eligible-block count of the result; may be NULL
 *   ws          scratch of bimask_refine_workspace_bytes(I, M, rounds) bytes
 * rounds == 0 only counts.  N <= 4 (N <= 2 at M = 4), I even, I < 2^24. */
size_t bimask_refine_workspace_bytes(int I, int M, int rounds);
int bimask_perm_refine(const uint32_t* maskbits_f, int I, int J, int N, int M, int rounds, uint64_t seed,
                       int32_t* perm_inout, int64_t* count_out, void* ws, size_t ws_bytes, void* stream);

/* The backward mask with another criterion for choosing the N survivors of a column block (the
 * ablation on binarization criteria, Sec. 4.4 / Table 8, compares these with Eq. 11's weight
 * magnitude).  As in Eq. 11, only entries whose forward bit is set compete, blocks are M
 * consecutive rows of the permuted matrix, and a block with at most N competitors keeps them all.
 *   BIMASK_CRIT_WEIGHT       Eq. 11; identical to bimask_bwd_mask.
 *   BIMASK_CRIT_SCORE        rank by |S| instead of |W| (S: device float[I*J], original row order;
 *                            S = the weight gradient of the previous iteration gives the
 *                            gradient-magnitude variant); ties to the lower row of the block.
 *   BIMASK_CRIT_MULTINOMIAL  N draws without replacement, each proportional to |w| among the
 *                            remaining competitors: u = 24 random bits from (seed, draw, block),
 *                            the draw takes the first remaining competitor whose running sum of
 *                            |w| (row order) exceeds u * total, else the lowest remaining one;
 *                            float32, every operation rounded once.
 *   BIMASK_CRIT_RANDOM       rank by a hashed 31-bit key of (seed, i*J + j): a uniformly random
 *                            N-subset of the competitors.
 * S may be NULL unless the criterion is SCORE; seed is ignored by WEIGHT and SCORE.  Everything
 * else (outputs, packing rules, alignment, errors) as for bimask_bwd_mask.  The variants run one
 * generic kernel for every M; only Eq. 11 has the tuned M = 4 kernels. */
enum { BIMASK_CRIT_WEIGHT = 0, BIMASK_CRIT_SCORE = 1, BIMASK_CRIT_MULTINOMIAL = 2, BIMASK_CRIT_RANDOM = 3 };
int bimask_bwd_mask_criterion(const float* W, const float* S_or_null, const uint32_t* maskbits_f,
                              const int32_t* perm, int I, int J, int N, int M, int criterion, uint64_t seed,
                              uint32_t* maskbits_b, uint16_t* vals_b, uint32_t* meta_b, void* hw_meta_b,
                              void* stream);

/* Eq. 3: Y[t, i] = sum_j X[t, j] (B * W)[i, j].  bf16 operands, fp32 accumulation, Y T x I bf16
 * (round to nearest even).  vals_f / hw_meta_f as written by bimask_fwd_mask. */
int bimask_spmm_fwd(const uint16_t* X, const uint16_t* vals_f, const void* hw_meta_f,
                    int T, int I, int J, uint16_t* Y, int32_t* status_word, void* stream);

/* Eq. 10: dX = (B-bar * W[perm,:])^T applied to dY[:, perm]; dX T x J bf16.
 *   ws: scratch (holds the column-permuted copy of dY, T x I bf16). */
int bimask_spmm_dgrad(const uint16_t* dY, const int32_t* perm, const uint16_t* vals_b,
                      const void* hw_meta_b, int T, int I, int J, uint16_t* dX,
                      void* ws, size_t ws_bytes, int32_t* status_word, void* stream);

/* Straight-through weight gradient (Sec. 3.1): dW[i, j] = sum_t dY[t, i] X[t, j], dense,
 * unmasked, fp32 I x J. */
int bimask_wgrad(const uint16_t* dY, const uint16_t* X, int T, int I, int J, float* dW,
                 void* ws, size_t ws_bytes, int32_t* status_word, void* stream);

/* One iteration of Alg. 1 for one layer (without the optimizer update): fwd mask + pack, sparse
 * forward, [search if do_search], bwd mask + pack, sparse input gradient, dense weight
 * gradient.  The caller sees one ordered step on `stream`: everything the call enqueues starts after the work
 * already on `stream` and is complete, as far as `stream` is concerned, when the work enqueued after the call starts.
 * Inside, layers between 1 and 100 GFLOP (2 T I J) run on four library-owned streams that fork from and join
 * `stream` by events: the dependent chain (masks, count, input gradient) and candidate generation + permutation of dY
 * on two streams of the highest priority, the weight gradient and the forward product on two of the lowest; the
 * first such call of a host thread on a device creates those streams and events (make it before any stream
 * capture; later calls can be captured, forks and joins included).
 * When the search is skipped, perm is used as given.  Limits: I <= 51200 (column permute of dY); with do_search
 * 1 <= P <= 65535, and I < 2^24 when the candidates are generated. */
typedef struct {
  int T, I, J, N, M, P;
  uint64_t seed;
  int do_search;              /* 0: use perm as given; 1: search and overwrite perm */
  const float* W;             /* I x J */
  const uint16_t* X;          /* T x J bf16 */
  const uint16_t* dY;         /* T x I bf16 */
  const int32_t* cands;       /* P x I or NULL (generate from seed) */
  int32_t* perm;              /* I, in/out */
  int32_t* best_idx;          /* 1 */
  int64_t* counts;            /* P */
  uint32_t* maskbits_f; uint16_t* vals_f; uint32_t* meta_f; void* hw_meta_f;
  uint32_t* maskbits_b; uint16_t* vals_b; uint32_t* meta_b; void* hw_meta_b;
  uint16_t* Y;                /* T x I bf16 */
  uint16_t* dX;               /* T x J bf16 */
  float* dW;                  /* I x J fp32 */
  void* ws; size_t ws_bytes;
  int32_t* status_word;
  void* stream;
} bimask_layer_args;

int bimask_layer_step(const bimask_layer_args* args);

/* The optimizer update that ends the loop body of Algorithm 1, fused with the first line
 * of the next iteration (forward mask, Eq. 4): one pass that reads W, dW and the momentum buffer,
 * writes the updated W and momentum, and emits the forward mask / 2:4 operand of the UPDATED
 * weights -- so an iteration that follows needs no bimask_fwd_mask of its own.
 *
 *   g = dW + weight_decay * W ;  mom = momentum * mom + g ;  W = W - lr * mom
 *
 * in float32, every product and sum rounded once in exactly that order (no fused multiply-add):
 * the updated weight decides mask bits, so the operation order is part of the contract.  The
 * straight-through estimator (Sec. 3.1) sends the gradient to all of W, masked or not.
 *   W, dW: device float[I*J]; W is updated in place.  mom: device float[I*J], updated in place;
 *   NULL means "no momentum buffer": it is read as zero and not stored (use with momentum == 0).
 *   Mask outputs as for bimask_fwd_mask (the same rules for patterns that do not pack).  M == 4 runs as one kernel; M in {8, 16} as an update pass followed
 *   by the mask kernel.  All pointers 16-byte aligned.  Errors as for bimask_fwd_mask. */
int bimask_sgd_fwd_mask(float* W, const float* dW, float* mom_or_null, int I, int J, int N, int M,
                        float lr, float momentum, float weight_decay,
                        uint32_t* maskbits_f, uint16_t* vals_f, uint32_t* meta_f, void* hw_meta_f, void* stream);

/* One whole iteration t of Algorithm 1 for one layer, including the Delta-T schedule of the search
 * and the optimizer update:
 *   1. forward mask of W (skipped when `premasked`: the previous call's step 6 already wrote it),
 *   2. Y (Eq. 3),
 *   3. if t % delta_t == 0: a new search, candidates drawn from seed + t / delta_t (each interval
 *      draws fresh candidates); otherwise layer.perm is used as it stands -- the caller sets it to
 *      the identity before the first call, and this call overwrites it whenever it searches,
 *   4. backward mask (Eq. 11), dX (Eq. 10), dense dW,
 *   5. (nothing: dW stays available to the caller),
 *   6. bimask_sgd_fwd_mask: W and mom updated in place, forward mask / operand of the new W written
 *      to layer.maskbits_f / vals_f / meta_f / hw_meta_f.
 * `layer` is read as by bimask_layer_step, except that do_search and seed are replaced as in step
 * 3 and that W is written.  After the last iteration vals_f / meta_f hold B.W of the final weights:
 * the algorithm's return value (for a pattern that does not pack: vals_f alone, dense). */
typedef struct bimask_train_args {
  bimask_layer_args layer;
  float* mom;              /* device float[I*J] or NULL (see bimask_sgd_fwd_mask) */
  float lr, momentum, weight_decay;
  int64_t t;               /* iteration number, counted from 1 as in Algorithm 1 */
  int32_t delta_t;         /* >= 1 */
  int32_t premasked;       /* non-zero: the forward mask of the current W is already in place */
} bimask_train_args;

int bimask_train_step(const bimask_train_args* args);

/* The layer step for a 3x3 convolution (zero padding 1, stride 1 or 2) on NHWC activations -- the
 * ResNet layers the paper trains.  The paper's W is the I x J matrix view of the filter with
 * J = 9*C and column j = (kh*3 + kw)*C + c (flatten order: the paper does not state one; this
 * keeps the channel index contiguous as in the activations), so masks, search and backward mask
 * are those of bimask_layer_step on that matrix.  The three products are convolutions:
 *   y [n,h,w,i] = sum_{kh,kw,c} x [n,h+kh-1,w+kw-1,c] (B.W)[i,(kh,kw,c)]                      (Eq. 3)
 *   dx[n,h,w,c] = sum_{kh,kw,i} dy[n,h-kh+1,w-kw+1,i] (B-bar.W[perm])...[i,(kh,kw,c)]         (Eq. 10)
 *   dW[i,(kh,kw,c)] = sum_{n,h,w} dy[n,h,w,i] x[n,h+kh-1,w+kw-1,c]                  (dense, Sec. 3.1)
 * (written for stride 1; with stride s the input pixel of tap (kh, kw) of output pixel (ho, wo) is
 * (ho*s + kh - 1, wo*s + kw - 1) and the output is Ho x Wo with Ho = (H - 1) / s + 1, Wo likewise).
 * `layer` is filled as for bimask_layer_step with T = NB*Ho*Wo (output pixels) and J = 9*C, except that
 *   layer.X  = x,  bf16 NB x H x W x C      (not T x J),
 *   layer.dX = dx, bf16 NB x H x W x C      (out),
 *   layer.dY = dy and layer.Y = y, bf16 NB x Ho x Wo x I (the same memory layout as T x I),
 *   layer.ws holds bimask_conv_workspace_bytes(...) bytes.
 * mode: BIMASK_CONV_EXPLICIT unfolds x into the T x 9C column matrix, runs the linear-layer
 * products and folds the column-space input gradient back (sum of the nine shifts, fp32);
 * BIMASK_CONV_IMPLICIT never builds the column matrix: the GEMM kernels fetch shifted pixel
 * patches with 4-D tensor loads (out-of-image pixels read as zero); BIMASK_CONV_AUTO takes the
 * implicit form for every product whose shape allows it (C % 64 == 0; the input gradient needs
 * C == 64 or C % 128 == 0; patterns with a 2:4 form) when the column matrix would
 * exceed 16 MiB and an output image has more than 64 pixels, and the explicit form otherwise.  Stride 2: the forward
 * product and the weight gradient take every second pixel in their tensor loads; the input gradient runs as four
 * stride-1 products, one per parity class (h % 2, w % 2) of the input pixels, each over the filter taps that reach
 * that class (one, two, two and four of the nine).  IMPLICIT needs C % 64 == 0 and a pattern with a 2:4 form; an
 * input gradient whose C is neither 64 nor a multiple of 128 keeps the explicit form then.  Otherwise IMPLICIT returns
 * BIMASK_EUNSUPPORTED.  C % 32 == 0 and I % 32 == 0 always.  The two forms round the
 * input gradient differently (explicit: nine bf16 partial results summed in fp32; implicit: one
 * fp32 accumulation), both within the products' tolerance. */
enum { BIMASK_CONV_AUTO = 0, BIMASK_CONV_EXPLICIT = 1, BIMASK_CONV_IMPLICIT = 2 };
typedef struct bimask_conv_args {
  bimask_layer_args layer;
  int NB, H, W, C;
  int mode;
  int stride;               /* 1 or 2 */
} bimask_conv_args;
size_t bimask_conv_workspace_bytes(int NB, int H, int W, int C, int I, int P, int stride);
int bimask_conv_layer_step(const bimask_conv_args* args);

/* The same step for a caller whose data lives in HOST memory (pinned memory recommended):
 * copies W, X, dY (and perm when do_search == 0, cands when given) to the device buffers named
 * in `dev`, runs bimask_layer_step there and copies Y, dX, dW, perm, best_idx, counts, the mask
 * bits and the status word back into the host buffers named in `host`; pointer fields of `host`
 * that are NULL are skipped.  `dev` must be fully populated; its sizes / flags are used, those of
 * `host` are ignored.
 *   bimask_layer_step_host        returns when the results are in host memory.
 *   bimask_layer_step_host_async  only enqueues: uploads, the step and downloads run on three
 *       queues (two copy streams owned by the library -- created with their events on the first
 *       call on a device, so make that call before any stream capture -- and `dev->stream`).  The
 *       library remembers the device buffers of the last four calls and orders a new call only
 *       behind earlier calls it shares device buffers with: a caller that alternates between two
 *       or more sets of device buffers gets the upload of one call, the kernels of another and the
 *       download of a third running at the same time (PCIe is full duplex); re-using one set
 *       serialises upload -> kernels -> download -> next upload, which is always correct.
 *       The host buffers of a call must stay valid and untouched until bimask_host_sync() (or a
 *       later blocking call) has returned.  Work the caller enqueues on dev->stream afterwards is
 *       ordered after this call's kernels but NOT after its downloads: do not overwrite the device
 *       outputs with other work before bimask_host_sync().  The host-buffer entry points keep
 *       per-device state (copy streams, the record of recent calls): call them from one host
 *       thread per device at a time.  The device-pointer entry points have no such state. */
int bimask_layer_step_host(const bimask_layer_args* dev, const bimask_layer_args* host,
                           int32_t* host_status_word);
int bimask_layer_step_host_async(const bimask_layer_args* dev, const bimask_layer_args* host,
                                 int32_t* host_status_word);
/* Waits for every download enqueued so far by the host-buffer entry points on the current device. */
int bimask_host_sync(void);

/* The same search for a caller that cannot hand over a workspace.  (No counterpart in the paper:
 * this entry point exists only because of how some programs manage GPU memory.)
 *
 * bimask_perm_search keeps the P x I generated candidates in `ws`, which somebody has to
 * allocate.  Some users of this library are not in a position to do that at the moment they call:
 * an inference or training runtime that has handed every byte of device memory to its own pool,
 * a plug-in that is only lent device pointers by its host application, or code running at a
 * point where calling the CUDA allocator is forbidden (it may synchronise the device).  For them
 * the candidates live in an 8 MiB array that is part of the library's device image, so this call
 * allocates nothing and asks for no scratch: it performs no cudaMalloc, no cudaFree and no
 * allocating library call.  Every GPU that loads the library carries those 8 MiB until exit.
 *
 *   - Limit: P * I <= bimask_perm_search_static_max_entries() (2 Mi entries, e.g. P = 128 at
 *     I = 16384); beyond that the call returns BIMASK_EUNSUPPORTED and launches nothing.
 *     Candidates are always generated from `seed` (same generator as bimask_perm_search with
 *     cands_or_null == NULL, so the results are identical).
 *   - The first call on each device looks up the array's device address (the current device must
 *     be the one `stream` belongs to); make that first call before any stream capture begins.
 *   - All calls share the one array and it keeps whatever the last call left there.  Nothing in
 *     it needs to start at zero (each call rewrites every entry it later reads), but two calls
 *     whose kernels overlap on the GPU -- different streams, or different host threads -- race
 *     on it: serialise them.
 *   - Inputs, outputs, alignment, return codes: as for bimask_perm_search, except that only M = 4
 *     (N = 1 or 2) is implemented here: other M return BIMASK_EUNSUPPORTED. */
int bimask_perm_search_static(const uint32_t* maskbits_f, int I, int J, int N, int M, int P, uint64_t seed,
                              int32_t* best_perm, int32_t* best_idx, int64_t* counts, void* stream);
size_t bimask_perm_search_static_max_entries(void);

/* Debug helper, not on the hot path: exercises the bounded wait that every tensor-core kernel
 * uses on its mbarriers.  One thread waits about a millisecond on a barrier nothing completes; the
 * wait gives up, *status_word (device int) becomes BIMASK_ETIMEOUT and the kernel returns
 * normally (no trap: the context stays usable). */
int bimask_debug_wait_probe(int32_t* status_word, void* stream);

/* Debug build (libbimask_debug.so, compiled with -DBIMASK_DEBUG): every kernel that turns a caller-supplied row
 * index (an entry of perm or of a candidate) into an address checks it against I.  Both builds clamp a bad index
 * into range, so nothing can fault; the debug build also records the first offender.  This call waits for the
 * device, then writes to the HOST array out[4] = {BIMASK_EBOUNDS or 0, site, index, bound} (site: 1 backward mask,
 * 2 count kernel, 3 column permute of dY, 4 / 5 the M = 8, 16 kernels' perm / candidate reads) and clears the
 * record.  In the release build it returns BIMASK_EUNSUPPORTED and out is all zero. */
int bimask_debug_status(int32_t* out);

/* Debug helper, not on the hot path: the candidate generator alone, cands (P x I i32) = the candidates
 * bimask_perm_search would generate from `seed`.  part_cap > 0 runs the part-wise generator (the one used
 * for I > 16384) with at most part_cap keys per sorting pass, which forces the multi-pass path that a part
 * takes when it draws more keys than its buffer holds; the result must not depend on part_cap. */
int bimask_debug_gen_candidates(uint64_t seed, int P, int I, int part_cap, int32_t* cands, void* stream);

/* Debug helper, not on the hot path: sets *ok (device int) to 1 iff each of the P rows of
 * cands is a permutation of 0..I-1.  ws: at least P * I bytes of scratch. */
int bimask_check_perms(const int32_t* cands, int P, int I, int32_t* ok, void* ws, size_t ws_bytes,
                       void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BIMASK_H */
