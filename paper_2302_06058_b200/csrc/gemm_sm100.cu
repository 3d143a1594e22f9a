// The three products of the layer step on the 5th-generation tensor cores:
//   sparse forward    D[i, t] = sum_j A_f[i, j] X[t, j]        (Eq. 3;  A_f 2:4 along j)
//   sparse input grad D[l, t] = sum_k A'[l, k] dYp[t, k]       (Eq. 10; A' 2:4 along permuted k)
//   dense weight grad D[i, j] = sum_t dY[t, i] X[t, j]         (straight-through estimator)
//
// One warp-specialised kernel template: a TMA producer thread fills a ring of shared-memory
// stages (operands in the 128-byte-swizzled layouts the tensor core reads directly), one thread
// issues tcgen05.mma (.sp for the 2:4 operand, whose index metadata is copied shared -> tensor
// memory with tcgen05.cp right before the MMAs that use it), accumulators live in tensor
// memory, and four epilogue warps drain them with tcgen05.ld and store the result.
//
// Every wait on an mbarrier carries a cycle budget: when it runs out the kernel writes
// BIMASK_ETIMEOUT to the caller's status word, all roles unwind, tensor memory is released and
// the kernel returns.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include <cuda_bf16.h>
#include <mutex>

namespace bimask {

namespace {

constexpr long long WAIT_BUDGET = 4000000000ll;      // ~2 s of SM clocks
constexpr int GEMM_THREADS = 192;                    // warp 0 TMA, warp 1 MMA, warps 2-5 epilogue

template <bool SPARSE, int N_TILE, int STAGES>
struct Cfg {
  static constexpr int M_TILE = 128;
  static constexpr int K_TILE = SPARSE ? 128 : 64;               // logical reduction elements per stage
  static constexpr int A_BYTES = 16384;                          // 128 x 64 bf16 either way
  static constexpr int B_BYTES = N_TILE * K_TILE * 2;
  static constexpr int E_BYTES = SPARSE ? 2048 : 0;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + E_BYTES;
  static constexpr int META_COLS = SPARSE ? 4 : 0;
  static constexpr int TMEM_COLS = (N_TILE + META_COLS) <= 128 ? 128 : (N_TILE + META_COLS) <= 256 ? 256 : 512;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
};

struct GemmParams {
  const uint8_t* hw_meta;   // sparse only
  int tiles_k_meta;         // number of 128-wide k tiles in the metadata image
  int Mdim, Ndim, Kdim;     // D is Mdim x Ndim, reduction length Kdim (logical)
  int k_tiles_per_split;    // dense split-K: k tiles handled by one blockIdx.z
  void* out;                // sparse: bf16 [Ndim][Mdim];  dense: fp32 [split][Mdim][Ndim]
  int32_t* status_word;
};

template <bool SPARSE, int N_TILE, int STAGES>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmapA, const __grid_constant__ CUtensorMap tmapB,
            const GemmParams p) {
  using C = Cfg<SPARSE, N_TILE, STAGES>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bar_base = base + STAGES * C::STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  const uint32_t tmem_full_bar = bar_base + 8u * (2 * STAGES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(base_ptr + STAGES * C::STAGE_BYTES + 8 * (2 * STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * C::M_TILE;
  const int n0 = blockIdx.y * N_TILE;
  const int k_tiles_total = (p.Kdim + C::K_TILE - 1) / C::K_TILE;
  const int kt_begin = blockIdx.z * p.k_tiles_per_split;
  const int kt_end = min(k_tiles_total, kt_begin + p.k_tiles_per_split);
  const int num_kt = kt_end - kt_begin;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    ptx::mbar_init(tmem_full_bar, 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmapA);
    ptx::prefetch_tmap(&tmapB);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(tmem_slot), C::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_meta = tmem_base + N_TILE;     // 4 columns after the accumulator (multiple of 4)

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (ptx::elect_one()) {
      for (int it = 0; it < num_kt; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
        if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; break; }
        const int kt = kt_begin + it;
        const uint32_t a_s = base + s * C::STAGE_BYTES;
        const uint32_t b_s = a_s + C::A_BYTES;
        ptx::mbar_expect_tx(full_bar(s), C::STAGE_BYTES);
        if (SPARSE) {
          ptx::tma_load_2d(a_s, &tmapA, kt * 64, m0, full_bar(s));                      // 64 compressed x 128 rows
          ptx::tma_load_2d(b_s, &tmapB, kt * 128, n0, full_bar(s));                     // k 0..63
          ptx::tma_load_2d(b_s + N_TILE * 128, &tmapB, kt * 128 + 64, n0, full_bar(s)); // k 64..127
          ptx::bulk_load(b_s + C::B_BYTES,
                         p.hw_meta + ((size_t)blockIdx.x * p.tiles_k_meta + kt) * 2048, 2048, full_bar(s));
        } else {
#pragma unroll
          for (int b = 0; b < 2; ++b) ptx::tma_load_2d(a_s + b * 8192, &tmapA, m0 + 64 * b, kt * 64, full_bar(s));
#pragma unroll
          for (int b = 0; b < N_TILE / 64; ++b) ptx::tma_load_2d(b_s + b * 8192, &tmapB, n0 + 64 * b, kt * 64, full_bar(s));
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (ptx::elect_one()) {
      constexpr uint32_t idesc = ptx::idesc_bf16(128, N_TILE, !SPARSE, !SPARSE, SPARSE);
      bool ok = true;
      for (int it = 0; it < num_kt && ok; ++it) {
        const int s = it % STAGES;
        const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
        if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, WAIT_BUDGET)) { *abort_flag = 1; ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t a_s = base + s * C::STAGE_BYTES;
        const uint32_t b_s = a_s + C::A_BYTES;
        if (SPARSE) {
          ptx::tmem_cp_128x128b(tmem_meta, ptx::smem_desc(b_s + C::B_BYTES, 0, 128, 0));
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t ad = ptx::smem_desc(a_s + kb * 32, 16, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + (kb >> 1) * (N_TILE * 128) + (kb & 1) * 64, 16, 1024, 2);
            ptx::mma_sparse(tmem_base, ad, bd, tmem_meta + (kb & ~1), idesc | (uint32_t)(kb & 1), (it | kb) != 0);
          }
        } else {
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint64_t ad = ptx::smem_desc(a_s + kb * 2048, 8192, 1024, 2);
            const uint64_t bd = ptx::smem_desc(b_s + kb * 2048, 8192, 1024, 2);
            ptx::mma_dense(tmem_base, ad, bd, idesc, (it | kb) != 0);
          }
        }
        ptx::tc_commit(empty_bar(s));
      }
      if (ok) ptx::tc_commit(tmem_full_bar);
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                               // TMEM lane quadrant this warp may read
    bool ok = true;
    if (num_kt > 0) ok = ptx::mbar_wait_bounded(tmem_full_bar, 0, abort_flag, WAIT_BUDGET);
    if (!ok) *abort_flag = 1;
    ptx::tc_fence_after();
    const int m = m0 + 32 * q + lane;
    if (ok) {
#pragma unroll 1
      for (int c = 0; c < N_TILE / 32; ++c) {
        uint32_t r[32];
        if (num_kt > 0) {
          ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(32 * q) << 16) + 32 * c, r);
          ptx::tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
        const int nb = n0 + 32 * c;
        if (SPARSE) {
          __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out);
          if (m < p.Mdim) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (nb + j < p.Ndim) out[(size_t)(nb + j) * p.Mdim + m] = __float2bfloat16_rn(__uint_as_float(r[j]));
          }
        } else {
          float* out = reinterpret_cast<float*>(p.out) + (size_t)blockIdx.z * p.Mdim * p.Ndim;
          if (m < p.Mdim && nb < p.Ndim) {          // Ndim % 32 == 0: a 32-column chunk is all in or all out
            float4* dst = reinterpret_cast<float4*>(out + (size_t)m * p.Ndim + nb);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                   __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status_word, (int32_t)BIMASK_ETIMEOUT);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------
// dY[:, perm]: a streaming pass, one CTA per token row chunk; the row is read coalesced into
// shared memory and written back permuted with 16-byte stores.
// ------------------------------------------------------------------------------------------
constexpr int PERMUTE_THREADS = 256;

__global__ void __launch_bounds__(PERMUTE_THREADS)
permute_cols_kernel(const uint16_t* __restrict__ dY, const int32_t* __restrict__ perm, int T, int I,
                    uint16_t* __restrict__ dYp) {
  extern __shared__ uint16_t row_s[];
  for (int t = blockIdx.x; t < T; t += gridDim.x) {
    const uint4* src = reinterpret_cast<const uint4*>(dY + (size_t)t * I);
    uint4* row4 = reinterpret_cast<uint4*>(row_s);
    for (int i = threadIdx.x; i < (I >> 3); i += PERMUTE_THREADS) row4[i] = __ldg(src + i);
    __syncthreads();
    uint4* dst = reinterpret_cast<uint4*>(dYp + (size_t)t * I);
    for (int i = threadIdx.x; i < (I >> 3); i += PERMUTE_THREADS) {
      const int4 pa = __ldg(reinterpret_cast<const int4*>(perm) + 2 * i);
      const int4 pb = __ldg(reinterpret_cast<const int4*>(perm) + 2 * i + 1);
      const int idx[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
      uint32_t v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const uint32_t lo = row_s[min(max(idx[2 * e], 0), I - 1)];
        const uint32_t hi = row_s[min(max(idx[2 * e + 1], 0), I - 1)];
        v[e] = lo | (hi << 16);
      }
      dst[i] = make_uint4(v[0], v[1], v[2], v[3]);
    }
    __syncthreads();
  }
}

// Sum of split-K partials: out[e] = sum_s part[s][e].
__global__ void splitk_reduce_kernel(const float4* __restrict__ part, int splits, long long n4,
                                     float4* __restrict__ out) {
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += (long long)gridDim.x * blockDim.x) {
    float4 acc = part[e];
    for (int s = 1; s < splits; ++s) {
      const float4 v = part[(long long)s * n4 + e];
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    out[e] = acc;
  }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  });
  return fn;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `outer` rows, box = 64 x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
int make_tmap(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  BIMASK_REQUIRE(fn != nullptr, BIMASK_ECUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  BIMASK_REQUIRE(r == CUDA_SUCCESS, BIMASK_ECUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return BIMASK_OK;
}

template <typename K>
int set_smem_attr(K kernel, int bytes) {
  BIMASK_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  return BIMASK_OK;
}

template <int N_TILE, int STAGES>
int run_sparse(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
               uint16_t* out, int32_t* status_word, cudaStream_t s) {
  using C = Cfg<true, N_TILE, STAGES>;
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap(&ta, vals, (uint64_t)Kdim / 2, (uint64_t)Mdim, 128)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, Bop, (uint64_t)Kdim, (uint64_t)Ndim, N_TILE)) != BIMASK_OK) return rc;
  auto kern = gemm_kernel<true, N_TILE, STAGES>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.hw_meta = reinterpret_cast<const uint8_t*>(hw_meta);
  p.tiles_k_meta = (Kdim + 127) / 128;
  p.Mdim = Mdim; p.Ndim = Ndim; p.Kdim = Kdim;
  p.k_tiles_per_split = (Kdim + 127) / 128;
  p.out = out;
  p.status_word = status_word;
  dim3 grid((Mdim + 127) / 128, (Ndim + N_TILE - 1) / N_TILE, 1);
  kern<<<grid, GEMM_THREADS, C::SMEM_BYTES, s>>>(ta, tb, p);
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace

int launch_spmm(const uint16_t* vals, const void* hw_meta, const uint16_t* Bop, int Mdim, int Ndim, int Kdim,
                uint16_t* out, int32_t* status_word, cudaStream_t s) {
  if (Ndim > 128) return run_sparse<256, 2>(vals, hw_meta, Bop, Mdim, Ndim, Kdim, out, status_word, s);
  return run_sparse<128, 4>(vals, hw_meta, Bop, Mdim, Ndim, Kdim, out, status_word, s);
}

int launch_permute_cols(const uint16_t* dY, const int32_t* perm, int T, int I, uint16_t* dYp, cudaStream_t s) {
  const size_t smem = (size_t)I * 2;
  static bool attr_done = false;
  if (!attr_done) {
    BIMASK_CUDA_OK(cudaFuncSetAttribute(permute_cols_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    attr_done = true;
  }
  int grid = T < 148 * 8 ? T : 148 * 8;
  permute_cols_kernel<<<grid, PERMUTE_THREADS, smem, s>>>(dY, perm, T, I, dYp);
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

// Split-K plan of the dense product, shared by the launcher and the workspace-size query.
void wgrad_plan(int T, int I, int J, int* n_tile, int* splits, int* k_tiles_per_split) {
  const int nt = 256;
  const int tiles = ((I + 127) / 128) * ((J + nt - 1) / nt);
  const int k_tiles = (T + 63) / 64;
  int sp = 1;
  if (tiles < 148) {
    sp = (2 * 148 + tiles - 1) / tiles;
    const int max_by_k = k_tiles / 8 > 0 ? k_tiles / 8 : 1;        // at least 8 k tiles per split
    if (sp > max_by_k) sp = max_by_k;
    if (sp > 64) sp = 64;
  }
  int per = (k_tiles + sp - 1) / sp;
  sp = (k_tiles + per - 1) / per;
  *n_tile = nt; *splits = sp; *k_tiles_per_split = per;
}

int launch_wgrad_impl(const uint16_t* dY, const uint16_t* X, int T, int I, int J, float* dW, float* partials,
                      int32_t* status_word, cudaStream_t s) {
  int nt, splits, per;
  wgrad_plan(T, I, J, &nt, &splits, &per);
  using C = Cfg<false, 256, 4>;
  CUtensorMap ta, tb;
  int rc;
  if ((rc = make_tmap(&ta, dY, (uint64_t)I, (uint64_t)T, 64)) != BIMASK_OK) return rc;
  if ((rc = make_tmap(&tb, X, (uint64_t)J, (uint64_t)T, 64)) != BIMASK_OK) return rc;
  auto kern = gemm_kernel<false, 256, 4>;
  if ((rc = set_smem_attr(kern, C::SMEM_BYTES)) != BIMASK_OK) return rc;
  GemmParams p;
  p.hw_meta = nullptr; p.tiles_k_meta = 0;
  p.Mdim = I; p.Ndim = J; p.Kdim = T;
  p.k_tiles_per_split = per;
  p.out = splits > 1 ? partials : dW;
  p.status_word = status_word;
  dim3 grid((I + 127) / 128, (J + nt - 1) / nt, splits);
  kern<<<grid, GEMM_THREADS, C::SMEM_BYTES, s>>>(ta, tb, p);
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  if (splits > 1) {
    const long long n4 = (long long)I * J / 4;
    long long blocks = (n4 + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    splitk_reduce_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(partials), splits, n4,
                                                         reinterpret_cast<float4*>(dW));
  count_launch();
    BIMASK_CUDA_OK(cudaGetLastError());
  }
  return BIMASK_OK;
}

}  // namespace bimask
