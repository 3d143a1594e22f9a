// Host side shared by the tensor-core kernels (tensor-map cache, SM count) and the two small kernels that go with
// the products: the column permutation of dY ahead of the input-gradient product, and the self-test of the bounded
// mbarrier wait.
#include "gemm_common.cuh"
#include <mutex>

namespace bimask {

namespace {

// ------------------------------------------------------------------------------------------
// dY[:, perm]: a streaming pass.  A CTA takes R token rows at a time (R = 4, or 2 for rows too
// long for a 4-row tile in shared memory): it reads
// them coalesced and stores them column-interleaved in shared memory (one 2R-byte word = the R
// rows' values of one column), so the gather costs one shared load per permuted column for all
// R rows; every thread then assembles eight consecutive permuted columns per row and writes
// them with one 16-byte store.
// ------------------------------------------------------------------------------------------
constexpr int PERMUTE_THREADS = 1024;

template <int R>
__global__ void __launch_bounds__(PERMUTE_THREADS)
permute_cols_kernel(const uint16_t* __restrict__ dY, const int32_t* __restrict__ perm, int T, int I,
                    uint16_t* __restrict__ dYp) {
  pdl_launch_dependents();
  pdl_wait();
  extern __shared__ uint32_t tile_w[];                   // R == 4: [I] x uint2, R == 2: [I] x uint32
  const int half = I >> 1;
  const int nthreads = (int)blockDim.x;                  // 256 .. 1024: short rows run more, smaller CTAs per SM
  for (int t0 = blockIdx.x * R; t0 < T; t0 += gridDim.x * R) {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(dY) + (size_t)t0 * half;
    // four column chunks per trip: 4 R loads in flight per thread before any is consumed
    for (int c0 = threadIdx.x; c0 < half; c0 += 4 * nthreads) {
      uint32_t r[4][R];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * nthreads;
#pragma unroll
        for (int j = 0; j < R; ++j) r[u][j] = (c < half && t0 + j < T) ? __ldg(src + (size_t)j * half + c) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * nthreads;
        if (c < half) {
          if (R == 4) {
            reinterpret_cast<uint4*>(tile_w)[c] =
                make_uint4(__byte_perm(r[u][0], r[u][1], 0x5410), __byte_perm(r[u][2], r[u][R - 1], 0x5410),
                           __byte_perm(r[u][0], r[u][1], 0x7632), __byte_perm(r[u][2], r[u][R - 1], 0x7632));
          } else {
            reinterpret_cast<uint2*>(tile_w)[c] =
                make_uint2(__byte_perm(r[u][0], r[u][1], 0x5410), __byte_perm(r[u][0], r[u][1], 0x7632));
          }
        }
      }
    }
    __syncthreads();
    for (int k8 = threadIdx.x; k8 < (I >> 3); k8 += nthreads) {
      const int4 pa = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8);
      const int4 pb = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8 + 1);
      const int idx[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
      uint32_t lo[8], hi[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int i = checked_row(idx[e], I, SITE_PERMUTE_PERM);
        if (R == 4) {
          const uint2 v = reinterpret_cast<const uint2*>(tile_w)[i];
          lo[e] = v.x; hi[e] = v.y;
        } else {
          lo[e] = tile_w[i]; hi[e] = 0u;
        }
      }
      uint4 o[4];
      o[0] = make_uint4(__byte_perm(lo[0], lo[1], 0x5410), __byte_perm(lo[2], lo[3], 0x5410),
                        __byte_perm(lo[4], lo[5], 0x5410), __byte_perm(lo[6], lo[7], 0x5410));
      o[1] = make_uint4(__byte_perm(lo[0], lo[1], 0x7632), __byte_perm(lo[2], lo[3], 0x7632),
                        __byte_perm(lo[4], lo[5], 0x7632), __byte_perm(lo[6], lo[7], 0x7632));
      o[2] = make_uint4(__byte_perm(hi[0], hi[1], 0x5410), __byte_perm(hi[2], hi[3], 0x5410),
                        __byte_perm(hi[4], hi[5], 0x5410), __byte_perm(hi[6], hi[7], 0x5410));
      o[3] = make_uint4(__byte_perm(hi[0], hi[1], 0x7632), __byte_perm(hi[2], hi[3], 0x7632),
                        __byte_perm(hi[4], hi[5], 0x7632), __byte_perm(hi[6], hi[7], 0x7632));
#pragma unroll
      for (int j = 0; j < R; ++j)
        if (t0 + j < T) reinterpret_cast<uint4*>(dYp + (size_t)(t0 + j) * I)[k8] = o[j];
    }
    __syncthreads();
  }
}

// Short rows (I <= 1024): a row is at most 2 KB and stays in L1, so each thread simply gathers
// its eight permuted columns from global memory; rows are spread over all threads.
__global__ void __launch_bounds__(256)
permute_cols_small_kernel(const uint16_t* __restrict__ dY, const int32_t* __restrict__ perm, long long T, int I,
                          uint16_t* __restrict__ dYp) {
  pdl_launch_dependents();
  pdl_wait();
  const int per_row = I >> 3;
  const long long total = T * per_row;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const long long t = e / per_row;
    const int k8 = (int)(e - t * per_row);
    const uint16_t* row = dY + t * I;
    const int4 pa = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8);
    const int4 pb = __ldg(reinterpret_cast<const int4*>(perm) + 2 * k8 + 1);
    const int idx[8] = {pa.x, pa.y, pa.z, pa.w, pb.x, pb.y, pb.z, pb.w};
    uint32_t v[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const uint32_t lo = __ldg(row + checked_row(idx[2 * h], I, SITE_PERMUTE_PERM));
      const uint32_t hi = __ldg(row + checked_row(idx[2 * h + 1], I, SITE_PERMUTE_PERM));
      v[h] = lo | (hi << 16);
    }
    reinterpret_cast<uint4*>(dYp + t * I)[k8] = make_uint4(v[0], v[1], v[2], v[3]);
  }
}

// Self-test of the bounded wait every GEMM role uses: one thread waits, with a budget of about
// a millisecond, on an mbarrier that nothing will ever complete.  The wait must give up, the kernel
// must report BIMASK_ETIMEOUT through the status word and return normally.
__global__ void wait_probe_kernel(long long budget_cycles, int32_t* __restrict__ status_word) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::fence_barrier_init();
    const bool ok = ptx::mbar_wait_bounded(ptx::smem_u32(&bar), 0, &abort_flag, budget_cycles);
    if (!ok) atomicExch(status_word, (int32_t)BIMASK_ETIMEOUT);
  }
}

}  // namespace

namespace {

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

// Encoding a tensor map costs a few microseconds on the host, which matters when a layer's
// kernels themselves run for ten.  A training loop passes the same buffers every step, so the
// encoded maps are kept in a small per-thread cache keyed by everything that went into them.
struct TmapKey {
  const void* ptr;
  uint64_t inner, outer, stride;
  uint32_t box_inner, box_outer;
  int dtype, swizzle;
  // rank 4 (NHWC activations: inner = channels, outer = W) when d2 != 0: extents H = d2, NB = d3,
  // densely packed (stride of H = W * stride, of NB = H * W * stride)
  uint64_t d2 = 0, d3 = 0;
  uint32_t box2 = 0, box3 = 0;
  uint32_t estride = 1;     // rank 4: traversal stride along W and H (the box spans estride * box pixels, takes `box`)
  bool operator==(const TmapKey& o) const {
    return ptr == o.ptr && inner == o.inner && outer == o.outer && stride == o.stride && box_inner == o.box_inner &&
           box_outer == o.box_outer && dtype == o.dtype && swizzle == o.swizzle && d2 == o.d2 && d3 == o.d3 &&
           box2 == o.box2 && box3 == o.box3 && estride == o.estride;
  }
};

int encode_cached(CUtensorMap* m, const TmapKey& key) {
  constexpr int SLOTS = 32;
  static thread_local TmapKey keys[SLOTS];
  static thread_local CUtensorMap maps[SLOTS];
  static thread_local bool used[SLOTS] = {false};
  static thread_local int next = 0;
  for (int i = 0; i < SLOTS; ++i)
    if (used[i] && keys[i] == key) { *m = maps[i]; return BIMASK_OK; }
  EncodeTiledFn fn = get_encode_fn();
  BIMASK_REQUIRE(fn != nullptr, BIMASK_ECUDA, "cuTensorMapEncodeTiled entry point not available");
  cuuint64_t dims[4] = {key.inner, key.outer, key.d2, key.d3};
  cuuint64_t strides[3] = {key.stride, key.stride * key.outer, key.stride * key.outer * key.d2};
  const cuuint32_t es = key.d2 ? key.estride : 1u;
  cuuint32_t box[4] = {key.box_inner, key.box_outer * es, key.box2 * es, key.box3};
  cuuint32_t estr[4] = {1, es, es, 1};
  CUresult r = fn(m, (CUtensorMapDataType)key.dtype, key.d2 ? 4 : 2, const_cast<void*>(key.ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, (CUtensorMapSwizzle)key.swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  BIMASK_REQUIRE(r == CUDA_SUCCESS, BIMASK_ECUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  keys[next] = key; maps[next] = *m; used[next] = true;
  next = (next + 1) % SLOTS;
  return BIMASK_OK;
}

}  // namespace

int sm_count() {
  static thread_local int cached_dev = -1, cached = 148;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev != cached_dev) {
    int n = 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess) { cached = n; cached_dev = dev; }
  }
  return cached;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `outer` rows, box = 64 x box_rows,
// 128-byte swizzle, out-of-range elements read as zero.
int make_tmap(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_rows) {
  return encode_cached(m, TmapKey{ptr, inner, outer, inner * 2, 64, box_rows, (int)CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                  (int)CU_TENSOR_MAP_SWIZZLE_128B});
}

// The metadata image as a 2-D tensor of u32: 256 words per row, two rows per 2048-byte block.
int make_tmap_meta(CUtensorMap* m, const void* ptr, uint64_t blocks) {
  return encode_cached(m, TmapKey{ptr, 256, blocks * 2, 1024, 256, 2, (int)CU_TENSOR_MAP_DATA_TYPE_UINT32,
                                  (int)CU_TENSOR_MAP_SWIZZLE_NONE});
}

// 4-D bf16 map of an NHWC tensor (channels, W, H, NB) for loads of 64-channel pixel boxes, 128-byte swizzle.
int make_tmap_nhwc_load(CUtensorMap* m, const void* ptr, int CH, int W, int H, int NB, int wb, int hb, int nb, int estride) {
  TmapKey k{ptr, (uint64_t)CH, (uint64_t)W, (uint64_t)CH * 2, 64, (uint32_t)wb, (int)CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
            (int)CU_TENSOR_MAP_SWIZZLE_128B};
  k.d2 = (uint64_t)H; k.d3 = (uint64_t)NB; k.box2 = (uint32_t)hb; k.box3 = (uint32_t)nb;
  k.estride = (uint32_t)estride;
  return encode_cached(m, k);
}

// fp32 result of the dense product, [planes][rows][inner] densely packed (planes = split-K partial sums), for stores
// of 32-column x 128-row boxes in the 128-byte-swizzled layout; rows and columns past the extents are clipped.
int make_tmap_f32_store(CUtensorMap* m, const void* ptr, uint64_t inner, uint64_t rows, uint64_t planes) {
  TmapKey k{ptr, inner, rows, inner * 4, 32, 128, (int)CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (int)CU_TENSOR_MAP_SWIZZLE_128B};
  k.d2 = planes; k.d3 = 1; k.box2 = 1; k.box3 = 1;
  return encode_cached(m, k);
}

// Generic 2-D tensor map without swizzle: `inner` contiguous elements of `elem_bytes` per row.
int make_tmap_plain(CUtensorMap* m, int dtype, const void* ptr, uint64_t inner, uint64_t outer, uint32_t box_inner,
                    uint32_t box_outer, uint32_t elem_bytes) {
  return encode_cached(m, TmapKey{ptr, inner, outer, inner * elem_bytes, box_inner, box_outer, dtype,
                                  (int)CU_TENSOR_MAP_SWIZZLE_NONE});
}

int launch_wait_probe(int32_t* status_word, cudaStream_t s) {
  BIMASK_CUDA_OK(launch_pdl(wait_probe_kernel, 1, 32, 0, s, 2000000ll, status_word));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

BIMASK_DEFINE_DEBUG_COLLECT(debug_collect_gemm_host)

int launch_permute_cols(const uint16_t* dY, const int32_t* perm, int T, int I, uint16_t* dYp, cudaStream_t s) {
  if (I <= 1024) {
    const long long total = (long long)T * (I >> 3);
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    BIMASK_CUDA_OK(launch_pdl(permute_cols_small_kernel, (unsigned)blocks, 256, 0, s, dY, perm, (long long)T, I, dYp));
    count_launch();
    BIMASK_CUDA_OK(cudaGetLastError());
    return BIMASK_OK;
  }
  if (int rc = set_smem_attr(permute_cols_kernel<4>, 200 * 1024)) return rc;
  if (int rc = set_smem_attr(permute_cols_kernel<2>, 200 * 1024)) return rc;
  const int R = (size_t)I * 8 <= 200 * 1024 ? 4 : 2;
  const size_t smem = (size_t)I * 2 * R;
  const int groups = (T + R - 1) / R;
  // a thread stages 16 row loads per trip and gathers 8 columns per trip: rows of I columns keep I / 8 threads busy
  const int threads = I >= 8192 ? PERMUTE_THREADS : I >= 4096 ? 512 : 256;
  int per_sm = (int)((200 * 1024) / smem);
  if (per_sm > 2048 / threads) per_sm = 2048 / threads;
  if (per_sm < 1) per_sm = 1;
  const int grid = groups < 148 * per_sm ? groups : 148 * per_sm;
  if (R == 4)
    BIMASK_CUDA_OK(launch_pdl(permute_cols_kernel<4>, grid, threads, smem, s, dY, perm, T, I, dYp));
  else
    BIMASK_CUDA_OK(launch_pdl(permute_cols_kernel<2>, grid, threads, smem, s, dY, perm, T, I, dYp));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace bimask
