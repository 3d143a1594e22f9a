// Shared host-side plumbing of the library: status codes, the per-thread error text and
// launch checking.  Device code in the other files includes this for the small bit helpers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdarg.h>
#include <atomic>
#include "../../include/bimask.h"

struct CUtensorMap_st;

namespace bimask {

void set_error(const char* fmt, ...);       // defined in api.cu
void count_launch(int n = 1);               // defined in api.cu: kernel launches made so far
int cuda_fail(cudaError_t e, const char* what);

#define BIMASK_CUDA_OK(call)                                   \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return ::bimask::cuda_fail(e__, #call); \
  } while (0)

#define BIMASK_REQUIRE(cond, code, ...)        \
  do {                                         \
    if (!(cond)) {                             \
      ::bimask::set_error(__VA_ARGS__);        \
      return (code);                           \
    }                                          \
  } while (0)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Programmatic dependent launch.  Every kernel of the library is launched with the attribute below, tells the
// runtime at its very start that the next kernel in the stream may be scheduled (pdl_launch_dependents) and
// waits for the kernels before it (pdl_wait) only after the part of its prologue that touches no global memory:
// barrier initialisation, tensor-memory allocation, table building.  So the launch latency and the prologue of a
// kernel overlap the tail of its predecessor; pdl_wait returns once the preceding grid has completed and its
// writes are visible, and since every kernel calls it, completion is transitive along the stream.
// Rule for kernel code: no global-memory access (read or write) before pdl_wait().
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

}  // namespace bimask

namespace bimask {

// The dynamic shared-memory limit of a kernel is set once per (device, kernel): the call costs a microsecond or two
// on the host, which a layer step of ten short launches would notice.  A kernel is always launched with the same size.
template <typename K>
inline int set_smem_attr(K kernel, int bytes) {
  constexpr int SLOTS = 64;
  static std::atomic<const void*> done[64][SLOTS];       // [device][slot]; zero-initialised
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = -1;
  const void* key = reinterpret_cast<const void*>(kernel);
  if (dev >= 0)
    for (int i = 0; i < SLOTS; ++i) {
      const void* seen = done[dev][i].load(std::memory_order_acquire);
      if (seen == key) return BIMASK_OK;
      if (seen == nullptr) break;
    }
  BIMASK_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  if (dev >= 0)
    for (int i = 0; i < SLOTS; ++i) {
      const void* expect = nullptr;
      if (done[dev][i].compare_exchange_strong(expect, key, std::memory_order_acq_rel) || expect == key) break;
    }
  return BIMASK_OK;
}

// Row indices that come from the caller (a permutation, a candidate) are clamped into range before they are used
// as addresses, so a bad entry can never fault a kernel.  In the debug build (-DBIMASK_DEBUG, libbimask_debug.so)
// the clamp also REPORTS: the first out-of-range index a kernel meets is recorded -- code BIMASK_EBOUNDS, a
// site number, the index and the bound -- in a small per-source-file device array that bimask_debug_status()
// collects.  Nothing traps; the release build compiles the record away.
#ifdef __CUDACC__
#ifdef BIMASK_DEBUG
namespace {
__device__ int tu_debug_record[4];                       // one per translation unit (internal linkage)
}
__device__ __forceinline__ int checked_row(int v, int n, int site) {
  if ((unsigned)v >= (unsigned)n) {
    if (atomicCAS(&tu_debug_record[0], 0, (int)BIMASK_EBOUNDS) == 0) {
      tu_debug_record[1] = site;
      tu_debug_record[2] = v;
      tu_debug_record[3] = n;
    }
    return v < 0 ? 0 : n - 1;
  }
  return v;
}
// host side of the same file: fetch and clear the record (synchronises the device)
#define BIMASK_DEFINE_DEBUG_COLLECT(name)                                                        \
  int name(int out[4]) {                                                                         \
    BIMASK_CUDA_OK(cudaDeviceSynchronize());                                                     \
    BIMASK_CUDA_OK(cudaMemcpyFromSymbol(out, tu_debug_record, 4 * sizeof(int)));                 \
    const int zero[4] = {0, 0, 0, 0};                                                            \
    BIMASK_CUDA_OK(cudaMemcpyToSymbol(tu_debug_record, zero, 4 * sizeof(int)));                  \
    return BIMASK_OK;                                                                            \
  }
#else
__device__ __forceinline__ int checked_row(int v, int n, int) {
  return (int)min((unsigned)max(v, 0), (unsigned)(n - 1));
}
#define BIMASK_DEFINE_DEBUG_COLLECT(name) \
  int name(int out[4]) { out[0] = out[1] = out[2] = out[3] = 0; return BIMASK_OK; }
#endif
#endif
// sites of checked_row, reported by bimask_debug_status
enum { SITE_BWD_MASK_PERM = 1, SITE_SCORE_CAND = 2, SITE_PERMUTE_PERM = 3, SITE_GENERIC_PERM = 4, SITE_GENERIC_CAND = 5 };
int debug_collect_mask(int out[4]);
int debug_collect_perm(int out[4]);
int debug_collect_gemm_host(int out[4]);
int debug_collect_generic(int out[4]);

// 2-D tensor map without swizzle (gemm_host.cu); dtype is a CUtensorMapDataType value.
int make_tmap_plain(CUtensorMap_st* m, int dtype, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_inner,
                    uint32_t box_outer, uint32_t elem_bytes);

// Launchers implemented in the .cu files (all enqueue on `s`, none synchronise).
// hw_meta_or_null: when given, the kernel also writes the tensor-core metadata image.  The 2:4 kernels (launch_fwd_mask,
// launch_sgd_fwd_mask, launch_bwd_mask) do so for any shape, padding included; the generic ones (M = 8, 16) only for
// operands without padding (rows and K multiples of 128): otherwise pass null and call launch_hw_meta afterwards.
int launch_fwd_mask(const float* W, int I, int J, int N, uint32_t* maskbits, uint16_t* vals,
                    uint32_t* meta, void* hw_meta_or_null, cudaStream_t s);
// forward mask of the weights after one SGD step, which the same kernel applies in place
int launch_sgd_fwd_mask(float* W, const float* dW, float* mom_or_null, int I, int J, int N, float lr, float momentum,
                        float weight_decay, uint32_t* maskbits, uint16_t* vals, uint32_t* meta,
                        void* hw_meta_or_null, cudaStream_t s);
int launch_hw_meta(const uint32_t* meta, int rows, int K, void* hw_meta, cudaStream_t s);
// 3x3 convolution, explicit form: x (NHWC) -> column matrix [T][9C]; column-space gradient -> dx (NHWC)
int launch_im2col3x3(const uint16_t* x, int NB, int H, int W, int C, int stride, uint16_t* cols, cudaStream_t s);
int launch_col2im3x3(const uint16_t* dcols, int NB, int H, int W, int C, int stride, uint16_t* dx, cudaStream_t s);
int launch_bwd_mask(const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                    int N, uint32_t* maskbits_b, uint16_t* vals_b, uint32_t* meta_b, void* hw_meta_or_null,
                    cudaStream_t s);
// zero_counts / zero_ticket (optional): the generator also zeroes counts[0..P) and *zero_ticket for the count kernel
// part_cap > 0 (debug): the part-wise generator with at most that many keys per sorting pass
int launch_gen_candidates(uint64_t seed, int P, int I, int32_t* cands, cudaStream_t s, int64_t* zero_counts = nullptr,
                          int32_t* zero_ticket = nullptr, int part_cap = 0);
// best_idx / best_perm (optional): fused pick by the kernel's last CTA; zeroed: counts and *best_idx are already zero
int launch_score(const uint32_t* maskbits_f, const int32_t* cands, int I, int J, int N, int P,
                 int64_t* counts, cudaStream_t s, bool zeroed = false, int32_t* best_idx = nullptr,
                 int32_t* best_perm = nullptr);
int launch_pick(const int64_t* counts, const int32_t* cands, int P, int I, int32_t* best_idx,
                int32_t* best_perm, cudaStream_t s);
// N:M patterns with M = 8 or 16 (nm_generic_kernels.cu); vals / meta may be null (mask bits only).
// mode (generic mask launchers): 0 mask bits only, 1 the 2:4 operand, 2 the dense masked bf16 operand in `vals`
// dW != nullptr: the optimizer update of Alg. 1 is applied to W (and mom_or_null) as the weights stream through.
int launch_fwd_mask_generic(const float* W, int I, int J, int N, int M, uint32_t* maskbits, uint16_t* vals_or_null,
                            uint32_t* meta_or_null, int mode, void* hw_meta_or_null, cudaStream_t s,
                            const float* dW = nullptr, float* mom_or_null = nullptr, float lr = 0.f, float momentum = 0.f,
                            float weight_decay = 0.f);
int launch_score_generic(const uint32_t* bits, const int32_t* cands, int I, int J, int N, int M, int P,
                         int64_t* counts, cudaStream_t s);
int launch_bwd_mask_generic(const float* W, const uint32_t* maskbits_f, const int32_t* perm, int I, int J, int N, int M,
                            uint32_t* maskbits_b, uint16_t* vals_b_or_null, uint32_t* meta_b_or_null, int mode,
                            void* hw_meta_or_null, cudaStream_t s);
int launch_bwd_mask_criterion(const float* W, const float* S, const uint32_t* maskbits_f, const int32_t* perm, int I, int J,
                              int N, int M, int crit, uint64_t seed, uint32_t* maskbits_b, uint16_t* vals_b_or_null,
                              uint32_t* meta_b_or_null, int mode, void* hw_meta_or_null, cudaStream_t s);
int launch_refine(const uint32_t* bits, int I, int J, int N, int M, int rounds, const int32_t* orders, int32_t* perm,
                  int32_t* gains, unsigned long long* block_best, cudaStream_t s);
int launch_check_perms(const int32_t* cands, int P, int I, int32_t* ok, uint8_t* seen, cudaStream_t s);
int launch_wait_probe(int32_t* status_word, cudaStream_t s);
int launch_permute_cols(const uint16_t* dY, const int32_t* perm, int T, int I, uint16_t* dYp, cudaStream_t s);
int launch_spmm(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
                uint16_t* out, int32_t* status_word, cudaStream_t s);
// 3x3 convolution products on shifted pixel boxes (no column matrix): mode 1 forward (tok = x, out = y with I
// channels), mode 2 input gradient (tok = permuted dy, out = dx with C channels); NHWC bf16 throughout.
// H x W is the INPUT image; stride 2 (forward only) gives an output of ((H-1)/2+1) x ((W-1)/2+1) pixels.
int launch_spmm_conv(int mode, const uint16_t* vals, const void* hw_meta, const uint16_t* tok, int NB, int H, int W, int C,
                     int I, int stride, uint16_t* out, int32_t* status_word, cudaStream_t s);
// Dense weight gradient of the 3x3 convolution on shifted pixel boxes; partials as sized by wgrad_conv_plan.
void wgrad_conv_plan(int NB, int H, int W, int C, int I, int stride, int* splits, int* k_tiles_per_split);
// reduce_stream / product_done: when given, the sum of the split-K partial results (if the plan has any) runs on
// reduce_stream behind the event product_done, which is recorded on s after the product kernel.
int launch_wgrad_conv(const uint16_t* dy, const uint16_t* x, int NB, int H, int W, int C, int I, int stride, float* dW,
                      float* partials, int32_t* status_word, cudaStream_t s, cudaStream_t reduce_stream = nullptr,
                      cudaEvent_t product_done = nullptr);
// Dense product for masked operands that do not fit the 2:4 format: out[n][m] = sum_k A[m][k] B[n][k],
// A bf16 [Mdim][Kdim], B bf16 [Ndim][Kdim], out bf16 [Ndim][Mdim] (same roles as launch_spmm).
int launch_dense_nt(const uint16_t* A, const uint16_t* Bop, int Mdim, int Ndim, int Kdim, uint16_t* out,
                    int32_t* status_word, cudaStream_t s);
void wgrad_plan(int T, int I, int J, int* n_tile, int* splits, int* k_tiles_per_split);
int launch_wgrad_impl(const uint16_t* dY, const uint16_t* X, int T, int I, int J, float* dW, float* partials,
                      int32_t* status_word, cudaStream_t s, cudaStream_t reduce_stream = nullptr,
                      cudaEvent_t product_done = nullptr);

}  // namespace bimask
