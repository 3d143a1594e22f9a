// 3x3 convolution layers (zero padding 1, stride 1 or 2, NHWC activations) for the layer step.
// The filter is the paper's I x J weight matrix with J = 9*C and column j = (kh*3 + kw)*C + c, so
// masks and search are unchanged.  This file holds the "explicit" form of the three products:
// the activations are unfolded into the T x 9C column matrix (T = NB*H*W pixels), the linear-layer
// kernels run on it, and the column-space input gradient is folded back (sum of the nine shifts).
// The implicit form (shifted tensor loads inside the GEMM kernels, no column matrix) lives with
// the GEMM kernels.
#include "common.cuh"

namespace bimask {

namespace {

// One thread per 16-byte chunk (eight channels) of the column matrix.
__global__ void im2col3x3_kernel(const uint4* __restrict__ x, int NB, int H, int W, int Ho, int Wo, int stride, int C8,
                                 long long total, uint4* __restrict__ cols) {
  pdl_launch_dependents();
  pdl_wait();
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c8 = (int)(idx % C8);
    long long r = idx / C8;
    const int khw = (int)(r % 9);
    r /= 9;                                              // output pixel index t = (n*Ho + ho)*Wo + wo
    const int wo = (int)(r % Wo);
    const long long nh = r / Wo;
    const int ho = (int)(nh % Ho);
    const long long n = nh / Ho;
    const int hs = ho * stride + khw / 3 - 1, ws = wo * stride + khw % 3 - 1;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (hs >= 0 && hs < H && ws >= 0 && ws < W) v = __ldg(x + ((n * H + hs) * W + ws) * C8 + c8);
    cols[idx] = v;
  }
}

__device__ __forceinline__ void add_bf16x2(float& lo, float& hi, uint32_t u) {
  lo += __uint_as_float(u << 16);
  hi += __uint_as_float(u & 0xFFFF0000u);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// dx[n, h, w, c] = sum over the nine taps of dXcol[(n, ho, wo), (kh*3+kw)*C + c] with ho*stride + kh - 1 = h and
// wo*stride + kw - 1 = w (taps with no such output pixel contribute nothing); fp32 sums.
__global__ void col2im3x3_kernel(const uint4* __restrict__ dcols, int NB, int H, int W, int Ho, int Wo, int stride, int C8,
                                 long long total, uint4* __restrict__ dx) {
  pdl_launch_dependents();
  pdl_wait();
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c8 = (int)(idx % C8);
    long long r = idx / C8;
    const int w = (int)(r % W);
    const long long nh = r / W;
    const int h = (int)(nh % H);
    const long long n = nh / H;
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
#pragma unroll
    for (int khw = 0; khw < 9; ++khw) {
      const int hn = h - khw / 3 + 1, wn = w - khw % 3 + 1;       // = ho * stride, wo * stride
      const int hs = hn / stride, ws = wn / stride;
      if (hn >= 0 && wn >= 0 && hs * stride == hn && ws * stride == wn && hs < Ho && ws < Wo) {
        const uint4 v = __ldg(dcols + (((n * Ho + hs) * Wo + ws) * 9 + khw) * C8 + c8);
        add_bf16x2(acc[0], acc[1], v.x);
        add_bf16x2(acc[2], acc[3], v.y);
        add_bf16x2(acc[4], acc[5], v.z);
        add_bf16x2(acc[6], acc[7], v.w);
      }
    }
    dx[idx] = make_uint4(pack_bf16x2(acc[0], acc[1]), pack_bf16x2(acc[2], acc[3]), pack_bf16x2(acc[4], acc[5]),
                         pack_bf16x2(acc[6], acc[7]));
  }
}

}  // namespace

int launch_im2col3x3(const uint16_t* x, int NB, int H, int W, int C, int stride, uint16_t* cols, cudaStream_t s) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  const long long total = (long long)NB * Ho * Wo * 9 * (C / 8);
  long long ctas = (total + 255) / 256;
  if (ctas > 148 * 16) ctas = 148 * 16;
  BIMASK_CUDA_OK(launch_pdl(im2col3x3_kernel, (unsigned)ctas, 256, 0, s, reinterpret_cast<const uint4*>(x), NB, H, W, Ho, Wo, stride, C / 8, total,
                                                  reinterpret_cast<uint4*>(cols)));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

int launch_col2im3x3(const uint16_t* dcols, int NB, int H, int W, int C, int stride, uint16_t* dx, cudaStream_t s) {
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  const long long total = (long long)NB * H * W * (C / 8);
  long long ctas = (total + 255) / 256;
  if (ctas > 148 * 16) ctas = 148 * 16;
  BIMASK_CUDA_OK(launch_pdl(col2im3x3_kernel, (unsigned)ctas, 256, 0, s, reinterpret_cast<const uint4*>(dcols), NB, H, W, Ho, Wo, stride, C / 8, total,
                                                  reinterpret_cast<uint4*>(dx)));
  count_launch();
  BIMASK_CUDA_OK(cudaGetLastError());
  return BIMASK_OK;
}

}  // namespace bimask
