// Minibatch objective on the device (the quantity whose gradient the sufficient factors carry, Section 3):
//   MLR  sum_i  logsumexp(z_i) - z_i[y_i]                         (cross-entropy of softmax(W x_i))
//   DML  sum_i  1/2 |z_i|^2 (similar pair)   or   1/2 max(0, margin - |z_i|^2) (dissimilar pair),  z_i = L d_i
//   SC   sum_i  1/2 |W a_i - x_i|^2
// One block per sample reduces its row of products in fp32 with a fixed combination order; the K per-sample
// values are then summed in fp64 by a single block, also in a fixed order, so the result is bit-reproducible.
// A monitoring helper: it is not part of the step and never touches W.
#include "common.cuh"

namespace sfb {
namespace {

__device__ __forceinline__ float warp_max_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <bool MAX>
__device__ float block_reduce(float v, float* red) {
  v = MAX ? warp_max_f(v) : warp_sum_f(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  const float r = (l < (int)(blockDim.x >> 5)) ? red[l] : (MAX ? -INFINITY : 0.f);
  return MAX ? warp_max_f(r) : warp_sum_f(r);
}

// rows: fp32, row i of the map; MLR and DML read z_i = W a_i, SC reads u_i = W a_i - x_i.
template <int MODEL>
__global__ void __launch_bounds__(256) sample_loss_kernel(RowMap rows, const int32_t* __restrict__ labels,
                                                          const uint8_t* __restrict__ similar, float margin, int K, int J,
                                                          float* __restrict__ loss_i, int* dev_status) {
  __shared__ float red[32];
  const int i = blockIdx.x;
  if (i >= K) return;
  const float* z = reinterpret_cast<const float*>(rows.row(i));
  float out;
  if (MODEL == SFB_MLR) {
    float m = -INFINITY;
    for (int j = threadIdx.x; j < J; j += 256) m = fmaxf(m, z[j]);
    m = block_reduce<true>(m, red);
    float s = 0.f;
    for (int j = threadIdx.x; j < J; j += 256) s += expf(z[j] - m);
    s = block_reduce<false>(s, red);
    const int y = labels[i];
    const bool bad = (y < 0) || (y >= J);
    if (bad && threadIdx.x == 0) atomicOr(dev_status, SFB_DEV_BAD_LABEL);
    out = bad ? 0.f : (m - z[y]) + logf(s);
  } else {
    float n = 0.f;
    for (int j = threadIdx.x; j < J; j += 256) n = fmaf(z[j], z[j], n);
    n = block_reduce<false>(n, red);
    if (MODEL == SFB_DML && similar[i] == 0) out = 0.5f * fmaxf(0.f, margin - n);
    else out = 0.5f * n;
  }
  if (threadIdx.x == 0) loss_i[i] = out;
}

__global__ void __launch_bounds__(1024) loss_total_kernel(const float* __restrict__ loss_i, int K, double* __restrict__ total) {
  __shared__ double part[1024];
  double acc = 0.0;
  for (int i = threadIdx.x; i < K; i += 1024) acc += (double)loss_i[i];
  part[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *total = part[0];
}

}  // namespace

int launch_sample_loss(cudaStream_t s, int model, RowMap rows, const int32_t* labels, const uint8_t* similar, float margin,
                       int K, int J, float* loss_i, double* total, int* dev_status) {
  if (model == SFB_MLR) sample_loss_kernel<SFB_MLR><<<K, 256, 0, s>>>(rows, labels, similar, margin, K, J, loss_i, dev_status);
  else if (model == SFB_DML) sample_loss_kernel<SFB_DML><<<K, 256, 0, s>>>(rows, labels, similar, margin, K, J, loss_i, dev_status);
  else sample_loss_kernel<SFB_SC><<<K, 256, 0, s>>>(rows, labels, similar, margin, K, J, loss_i, dev_status);
  loss_total_kernel<<<1, 1024, 0, s>>>(loss_i, K, total);
  return cudaGetLastError() == cudaSuccess ? 2 : SFB_ERR_CUDA;
}

}  // namespace sfb
