// Bandwidth-bound passes of the factor computation: the model epilogues that turn the products
// z_i = W a_i into the factor u_i, row copies, and the fp32 -> bf16 cast of W.
//
//   MLR  u_i = softmax(z_i) - onehot(y_i)   (chain rule on the multiclass logistic loss; Section 2.1)
//   DML  u_i = +z_i (similar pair) | -z_i * [|z_i|^2 < margin] (dissimilar pair)   (Section 2, DML)
//
// One thread block per sample row; the row is staged once in shared memory (when it fits) so HBM
// sees one read and one write per value; reductions over the J entries use warp shuffles.
#include "common.cuh"

namespace sfb {
namespace {

constexpr int ROW_CACHE_FLOATS = 48 * 1024;   // 192 KB of dynamic shared memory

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Block-wide reductions with a fixed combination order (bit-reproducible).
__device__ float block_max(float v, float* red) {
  v = warp_max(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float r = (l < (int)(blockDim.x >> 5)) ? red[l] : -INFINITY;
  return warp_max(r);
}
__device__ float block_sum(float v, float* red) {
  v = warp_sum(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) red[w] = v;
  __syncthreads();
  float r = (l < (int)(blockDim.x >> 5)) ? red[l] : 0.f;
  return warp_sum(r);
}

// Four products starting at column j: the sum, in split order, of the partial products of a reduction
// that the GEMM cut in `nsplit` ranges (partial s lives `stride` floats after partial s - 1).
__device__ __forceinline__ float4 ldz4(const float* zr, int j, int nsplit, long long stride) {
  float4 t = *reinterpret_cast<const float4*>(zr + j);
  for (int s = 1; s < nsplit; ++s) {
    const float4 q = *reinterpret_cast<const float4*>(zr + s * stride + j);
    t.x += q.x; t.y += q.y; t.z += q.z; t.w += q.w;
  }
  return t;
}

// Stores 4 consecutive values starting at column j (j % 4 == 0, j + 3 < ld).
__device__ __forceinline__ void store_u4(char* row, int j, float4 v, int es) {
  if (es == 4) {
    *reinterpret_cast<float4*>(row + (size_t)j * 4) = v;
  } else {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 p;
    p.x = *reinterpret_cast<uint32_t*>(&lo);
    p.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(row + (size_t)j * 2) = p;
  }
}

// z rows are fp32 with ld a multiple of 4; values beyond J inside the last float4 are ignored.
// SDCA (dual != nullptr; Section 2.1, "Stochastic DCA"): the factor is the damped dual step
// du_i = step * (dual_i + g_i) with g_i = softmax(z_i) - onehot(y_i), and dual_i <- dual_i - du_i in place
// (dual rows: fp32, ldd = J rounded up to 4 values per row, pad values written as zeros).
__device__ __forceinline__ float4 sdca_step4(float* dual_row, int j, int J, float4 g, float step, bool bad) {
  float4 d = *reinterpret_cast<const float4*>(dual_row + j);
  float4 du = make_float4(0.f, 0.f, 0.f, 0.f);
  if (!bad) {   // a sample with a bad label takes no step: its dual variables stay as they are
    du.x = step * (d.x + g.x); du.y = step * (d.y + g.y); du.z = step * (d.z + g.z); du.w = step * (d.w + g.w);
    d.x -= du.x; d.y -= du.y; d.z -= du.z; d.w -= du.w;
  }
  if (j + 1 >= J) { du.y = 0.f; d.y = 0.f; }
  if (j + 2 >= J) { du.z = 0.f; d.z = 0.f; }
  if (j + 3 >= J) { du.w = 0.f; d.w = 0.f; }
  *reinterpret_cast<float4*>(dual_row + j) = d;
  return du;
}

__global__ void __launch_bounds__(1024) finish_mlr_kernel(RowMap z, RowMap u, const int32_t* __restrict__ labels,
                                                                 int K, int J, int cache_floats, int* dev_status, int nsplit, long long zstride,
                                                                 float* __restrict__ dual, float sdca_step, CorrOut corr) {
  extern __shared__ __align__(16) float cache[];
  __shared__ float red[32];
  const int i = blockIdx.x;
  if (i >= K) return;
  const float* zr = reinterpret_cast<const float*>(z.row(i));
  char* ur = u.row(i);
  const int J4 = (J + 3) >> 2;
  const bool cached = (J4 * 4) <= cache_floats;
  const float kLog2e = 1.4426950408889634f;

  float m = -INFINITY;
  for (int q = threadIdx.x; q < J4; q += blockDim.x) {
    float4 t = ldz4(zr, q * 4, nsplit, zstride);
    const int j = q * 4;
    if (j + 1 >= J) t.y = -INFINITY;
    if (j + 2 >= J) t.z = -INFINITY;
    if (j + 3 >= J) t.w = -INFINITY;
    if (cached) *reinterpret_cast<float4*>(cache + j) = t;
    m = fmaxf(fmaxf(fmaxf(m, t.x), fmaxf(t.y, t.z)), t.w);
  }
  m = block_max(m, red);

  float s = 0.f;
  const float mb = m * kLog2e;
  for (int q = threadIdx.x; q < J4; q += blockDim.x) {
    const int j = q * 4;
    float4 t;
    if (cached) {
      t = *reinterpret_cast<const float4*>(cache + j);
    } else {
      t = ldz4(zr, j, nsplit, zstride);
      if (j + 1 >= J) t.y = -INFINITY;
      if (j + 2 >= J) t.z = -INFINITY;
      if (j + 3 >= J) t.w = -INFINITY;
    }
    t.x = exp2f(fmaf(t.x, kLog2e, -mb)); t.y = exp2f(fmaf(t.y, kLog2e, -mb));
    t.z = exp2f(fmaf(t.z, kLog2e, -mb)); t.w = exp2f(fmaf(t.w, kLog2e, -mb));
    if (cached) *reinterpret_cast<float4*>(cache + j) = t;
    s += (t.x + t.y) + (t.z + t.w);
  }
  s = block_sum(s, red);
  const float inv = 1.0f / s;

  const int y = labels[i];
  const bool bad = (y < 0) || (y >= J);
  if (bad && threadIdx.x == 0) atomicOr(dev_status, SFB_DEV_BAD_LABEL);
  const int ld4 = u.ld >> 2;   // u.ld is a multiple of 4 (fp32) or 8 (bf16)
  for (int q = threadIdx.x; q < ld4; q += blockDim.x) {
    const int j = q * 4;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q < J4 && !bad) {
      if (cached) {
        t = *reinterpret_cast<const float4*>(cache + j);
      } else {
        t = ldz4(zr, j, nsplit, zstride);
        t.x = exp2f(fmaf(t.x, kLog2e, -mb)); t.y = exp2f(fmaf(t.y, kLog2e, -mb));
        t.z = exp2f(fmaf(t.z, kLog2e, -mb)); t.w = exp2f(fmaf(t.w, kLog2e, -mb));
      }
      t.x *= inv; t.y *= inv; t.z *= inv; t.w *= inv;
      if (y == j) t.x -= 1.f;
      if (y == j + 1) t.y -= 1.f;
      if (y == j + 2) t.z -= 1.f;
      if (y == j + 3) t.w -= 1.f;
      if (j + 1 >= J) t.y = 0.f;
      if (j + 2 >= J) t.z = 0.f;
      if (j + 3 >= J) t.w = 0.f;
    }
    if (dual != nullptr && q < J4) t = sdca_step4(dual + (size_t)i * (J4 * 4), j, J, t, sdca_step, bad);
    store_u4(ur, j, t, u.es);
    if (corr.mn != nullptr) corr_store4(corr, i, u.B, j, t);
  }
}

__global__ void __launch_bounds__(1024) finish_dml_kernel(RowMap z, RowMap u, const uint8_t* __restrict__ similar,
                                                                 float margin, int K, int J, int cache_floats, int nsplit, long long zstride,
                                                                 uint8_t* __restrict__ active, CorrOut corr) {
  extern __shared__ __align__(16) float cache[];
  __shared__ float red[32];
  const int i = blockIdx.x;
  if (i >= K) return;
  const float* zr = reinterpret_cast<const float*>(z.row(i));
  char* ur = u.row(i);
  const int J4 = (J + 3) >> 2;
  const bool cached = (J4 * 4) <= cache_floats;

  float n = 0.f;
  for (int q = threadIdx.x; q < J4; q += blockDim.x) {
    float4 t = ldz4(zr, q * 4, nsplit, zstride);
    const int j = q * 4;
    if (j + 1 >= J) t.y = 0.f;
    if (j + 2 >= J) t.z = 0.f;
    if (j + 3 >= J) t.w = 0.f;
    if (cached) *reinterpret_cast<float4*>(cache + j) = t;
    n += (t.x * t.x + t.y * t.y) + (t.z * t.z + t.w * t.w);
  }
  n = block_sum(n, red);
  const bool sim = similar[i] != 0;
  const float g = sim ? 1.f : ((n < margin) ? -1.f : 0.f);   // strict hinge: inactive at equality
  if (active != nullptr && threadIdx.x == 0) active[i] = (g != 0.f) ? 1 : 0;   // u_i is all zeros otherwise

  const int ld4 = u.ld >> 2;
  for (int q = threadIdx.x; q < ld4; q += blockDim.x) {
    const int j = q * 4;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q < J4 && g != 0.f) {
      t = cached ? *reinterpret_cast<const float4*>(cache + j) : ldz4(zr, j, nsplit, zstride);
      t.x *= g; t.y *= g; t.z *= g; t.w *= g;
      if (j + 1 >= J) t.y = 0.f;
      if (j + 2 >= J) t.z = 0.f;
      if (j + 3 >= J) t.w = 0.f;
    }
    store_u4(ur, j, t, u.es);
    if (corr.mn != nullptr) corr_store4(corr, i, u.B, j, t);
  }
}

// Second half of the fused multiclass-logistic epilogue.  The forward GEMM left e[j] = exp(z[j] - m_p)
// in the u row (p = the half tile that holds class j) and (m_p, s_p = sum of those exps) per part.
// Here: m = max_p m_p, s = sum_p s_p exp(m_p - m), u[j] = e[j] * exp(m_p - m) / s - [j == label], in place.
template <int ES>
__global__ void __launch_bounds__(256) finish_mlr_fused_kernel(RowMap u, const float2* __restrict__ stats, int n_parts,
                                                               int part_cols, const int32_t* __restrict__ labels, int K,
                                                               int J, int* dev_status, float* __restrict__ dual,
                                                               float sdca_step) {
  extern __shared__ float scale[];   // [n_parts]
  __shared__ float red[32];
  const int i = blockIdx.x;
  if (i >= K) return;
  const float kLog2e = 1.4426950408889634f;
  const float2* st = stats + (size_t)i * n_parts;
  float m = -INFINITY;
  for (int q = threadIdx.x; q < n_parts; q += 256) m = fmaxf(m, st[q].x);
  m = block_max(m, red);
  float ssum = 0.f;
  for (int q = threadIdx.x; q < n_parts; q += 256) {
    const float2 ps = st[q];
    const float f = (ps.x == -INFINITY) ? 0.f : exp2f((ps.x - m) * kLog2e);
    scale[q] = f;
    ssum += ps.y * f;
  }
  ssum = block_sum(ssum, red);   // also orders the writes of scale[] before the reads below
  const float inv = 1.0f / ssum;
  const int y = labels[i];
  const bool bad = (y < 0) || (y >= J);
  if (bad && threadIdx.x == 0) atomicOr(dev_status, SFB_DEV_BAD_LABEL);
  char* ur = u.row(i);
  constexpr int PER = 16 / ES;          // values per 16-byte unit (part_cols is a multiple of it)
  const int units = u.ld / PER;
  for (int q = threadIdx.x; q < units; q += 256) {
    const int j = q * PER;
    uint4 raw = *reinterpret_cast<const uint4*>(ur + (size_t)q * 16);
    float vals[PER];
    if (ES == 4) {
      const float* f = reinterpret_cast<const float*>(&raw);
#pragma unroll
      for (int e = 0; e < PER; ++e) vals[e] = f[e];
    } else {
      const __nv_bfloat16* h = reinterpret_cast<const __nv_bfloat16*>(&raw);
#pragma unroll
      for (int e = 0; e < PER; ++e) vals[e] = __bfloat162float(h[e]);
    }
    const float f = (j < J && !bad) ? scale[j / part_cols] * inv : 0.f;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      float r = vals[e] * f;
      if (j + e == y) r -= 1.f;
      if (j + e >= J || bad) r = 0.f;
      vals[e] = r;
    }
    if (dual != nullptr && j < J) {   // SDCA: the factor becomes the dual step, the dual variables move by it
      float* drow = dual + (size_t)i * (((J + 3) >> 2) * 4);
#pragma unroll
      for (int e4 = 0; e4 < PER; e4 += 4) {
        if (j + e4 < J) {
          const float4 du = sdca_step4(drow, j + e4, J, make_float4(vals[e4], vals[e4 + 1], vals[e4 + 2], vals[e4 + 3]),
                                       sdca_step, bad);
          vals[e4] = du.x; vals[e4 + 1] = du.y; vals[e4 + 2] = du.z; vals[e4 + 3] = du.w;
        }
      }
    }
    if (ES == 4) {
      float* f4 = reinterpret_cast<float*>(&raw);
#pragma unroll
      for (int e = 0; e < PER; ++e) f4[e] = vals[e];
    } else {
      __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(&raw);
#pragma unroll
      for (int e = 0; e < PER; ++e) h[e] = __float2bfloat16_rn(vals[e]);
    }
    *reinterpret_cast<uint4*>(ur + (size_t)q * 16) = raw;
  }
}

// Unit-ball projection of the columns of W (sparse-coding prox).  One block owns 32 consecutive
// columns: 32 x 8 threads walk the rows (a warp reads one 128-byte line per row), the squared norms are
// combined in a fixed order, then the block rescales its columns (second read served by L2).  Columns
// with norm <= 1 are not written at all.
__global__ void __launch_bounds__(256) prox_unit_columns_kernel(float* __restrict__ W, int J, int D) {
  __shared__ float part[8][33];
  __shared__ float scale[32];
  const int c = threadIdx.x & 31, r = threadIdx.x >> 5;
  const int d = blockIdx.x * 32 + c;
  float acc = 0.f;
  if (d < D)
    for (int j = r; j < J; j += 8) {
      const float w = W[(size_t)j * D + d];
      acc = fmaf(w, w, acc);
    }
  part[r][c] = acc;
  __syncthreads();
  if (r == 0) {
    float n2 = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) n2 += part[q][c];
    scale[c] = (n2 > 1.0f) ? 1.0f / sqrtf(n2) : 1.0f;
  }
  __syncthreads();
  const float sc = scale[c];
  if (d < D && sc != 1.0f)
    for (int j = r; j < J; j += 8) W[(size_t)j * D + d] *= sc;
}

// 16-byte-vectorised row copy; rows are whole numbers of 16-byte units on both sides.
__global__ void __launch_bounds__(256) copy_rows_kernel(RowMap src, RowMap dst, int K, int cols, CorrOut corr) {
  const int units_dst = dst.ld * dst.es / 16;
  const int per = 16 / dst.es;
  const long long total = (long long)K * units_dst;
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < total;
       g += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(g / units_dst), q = (int)(g % units_dst);
    const int c = q * per;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (c < cols && c < src.ld) {
      val = *reinterpret_cast<const uint4*>(src.row(i) + (size_t)q * 16);
      if (c + per > cols) {   // mask the tail beyond `cols`
        if (dst.es == 4) {
          uint32_t* w = reinterpret_cast<uint32_t*>(&val);
          for (int e = 0; e < 4; ++e)
            if (c + e >= cols) w[e] = 0u;
        } else {
          uint16_t* h = reinterpret_cast<uint16_t*>(&val);
          for (int e = 0; e < 8; ++e)
            if (c + e >= cols) h[e] = 0;
        }
      }
    }
    *reinterpret_cast<uint4*>(dst.row(i) + (size_t)q * 16) = val;
    if (corr.mn != nullptr || corr.km != nullptr)   // fp32 rows only (the compensated path)
      corr_store4(corr, i, dst.B, c, make_float4(__uint_as_float(val.x), __uint_as_float(val.y), __uint_as_float(val.z),
                                                 __uint_as_float(val.w)));
  }
}

// v rows = Xa - Xb (one fp32 subtraction per element), pad columns zero; 4 values per thread.
__global__ void __launch_bounds__(256) diff_rows_kernel(const float* __restrict__ Xa, const float* __restrict__ Xb, RowMap v,
                                                        int K, int D, CorrOut corr) {
  const int units = v.ld >> 2;
  const long long total = (long long)K * units;
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < total;
       g += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(g / units), c = (int)(g % units) * 4;
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c + 3 < D && (D & 3) == 0) {
      const float4 a = *reinterpret_cast<const float4*>(Xa + (size_t)i * D + c);
      const float4 b = *reinterpret_cast<const float4*>(Xb + (size_t)i * D + c);
      r = make_float4(__fsub_rn(a.x, b.x), __fsub_rn(a.y, b.y), __fsub_rn(a.z, b.z), __fsub_rn(a.w, b.w));
    } else {
      float* e = reinterpret_cast<float*>(&r);
      for (int q = 0; q < 4; ++q)
        if (c + q < D) e[q] = __fsub_rn(Xa[(size_t)i * D + c + q], Xb[(size_t)i * D + c + q]);
    }
    *reinterpret_cast<float4*>(v.row(i) + (size_t)c * 4) = r;
    if (corr.mn != nullptr || corr.km != nullptr) corr_store4(corr, i, v.B, c, r);
  }
}

__global__ void __launch_bounds__(256) cast_bf16_kernel(const float* __restrict__ W, __nv_bfloat16* __restrict__ Wb,
                                                        long long n4) {
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < n4; g += (long long)gridDim.x * blockDim.x) {
    const float4 t = reinterpret_cast<const float4*>(W)[g];
    __nv_bfloat162 lo = __floats2bfloat162_rn(t.x, t.y), hi = __floats2bfloat162_rn(t.z, t.w);
    uint2 p;
    p.x = *reinterpret_cast<uint32_t*>(&lo);
    p.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(Wb)[g] = p;
  }
}

// Long rows take a whole SM's worth of shared memory, so one block must supply all the memory parallelism.
int fin_threads(int J) { return J >= 8192 ? 1024 : 256; }

int fin_cache_floats(int J) {
  const int need = ((J + 3) / 4) * 4;
  return need <= ROW_CACHE_FLOATS ? need : 0;
}

}  // namespace

int launch_finish_mlr(cudaStream_t s, RowMap z, RowMap u, const int32_t* labels, int K, int J, int* dev_status,
                      int nsplit, long long split_stride_bytes, float* dual, float sdca_step, CorrOut corr) {
  const int cf = fin_cache_floats(J);
  static PerDeviceOnce attr_once;   // function attributes are per device
  if (attr_once.first()) {
    cudaFuncSetAttribute(finish_mlr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ROW_CACHE_FLOATS * 4);
    cudaFuncSetAttribute(finish_dml_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ROW_CACHE_FLOATS * 4);
  }
  finish_mlr_kernel<<<K, fin_threads(J), (size_t)cf * 4, s>>>(z, u, labels, K, J, cf, dev_status, nsplit, split_stride_bytes / 4,
                                                              dual, sdca_step, corr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

// idx[0 .. n) = the samples i < K with active[i] != 0, in ascending order; *n_out = n.  One block, ordered.
__global__ void __launch_bounds__(1024) compact_active_kernel(const uint8_t* __restrict__ active, int K, int* __restrict__ idx,
                                                              int* __restrict__ n_out) {
  __shared__ int warp_cnt[32];
  __shared__ int base;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int start = 0; start < K; start += 1024) {
    const int i = start + threadIdx.x;
    const bool f = i < K && active[i] != 0;
    const unsigned m = __ballot_sync(0xffffffffu, f);
    const int before = __popc(m & ((1u << lane) - 1u));
    if (lane == 0) warp_cnt[warp] = __popc(m);
    __syncthreads();
    int off = 0;
    for (int w = 0; w < warp; ++w) off += warp_cnt[w];
    if (f) idx[base + off + before] = i;
    __syncthreads();
    if (threadIdx.x == 0) {
      int t = 0;
      for (int w = 0; w < 32; ++w) t += warp_cnt[w];
      base += t;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) *n_out = base;
}

int launch_compact_active(cudaStream_t s, const uint8_t* active, int K, int* idx, int* n_out) {
  compact_active_kernel<<<1, 1024, 0, s>>>(active, K, idx, n_out);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_finish_dml(cudaStream_t s, RowMap z, RowMap u, const uint8_t* similar, float margin, int K, int J,
                      int nsplit, long long split_stride_bytes, uint8_t* active, CorrOut corr) {
  const int cf = fin_cache_floats(J);
  static PerDeviceOnce attr_once;   // function attributes are per device
  if (attr_once.first()) {
    cudaFuncSetAttribute(finish_mlr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ROW_CACHE_FLOATS * 4);
    cudaFuncSetAttribute(finish_dml_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ROW_CACHE_FLOATS * 4);
  }
  finish_dml_kernel<<<K, fin_threads(J), (size_t)cf * 4, s>>>(z, u, similar, margin, K, J, cf, nsplit, split_stride_bytes / 4,
                                                              active, corr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_finish_mlr_fused(cudaStream_t s, RowMap u, const float2* stats, int n_parts, int part_cols,
                            const int32_t* labels, int K, int J, int* dev_status, float* dual, float sdca_step) {
  const size_t smem = (size_t)n_parts * sizeof(float);
  if (smem > 48 * 1024) return SFB_ERR_SHAPE;
  if (u.es == 4)
    finish_mlr_fused_kernel<4><<<K, 256, smem, s>>>(u, stats, n_parts, part_cols, labels, K, J, dev_status, dual, sdca_step);
  else
    finish_mlr_fused_kernel<2><<<K, 256, smem, s>>>(u, stats, n_parts, part_cols, labels, K, J, dev_status, dual, sdca_step);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_prox_unit_columns(cudaStream_t s, float* W, int J, int D) {
  prox_unit_columns_kernel<<<(D + 31) / 32, 256, 0, s>>>(W, J, D);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_copy_rows(cudaStream_t s, RowMap src, RowMap dst, int K, int cols, CorrOut corr) {
  const long long total = (long long)K * (dst.ld * dst.es / 16);
  if (total == 0) return 0;
  const int blocks = (int)((total + 255) / 256 < 148LL * 16 ? (total + 255) / 256 : 148LL * 16);
  copy_rows_kernel<<<blocks, 256, 0, s>>>(src, dst, K, cols, corr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_diff_rows(cudaStream_t s, const float* Xa, const float* Xb, RowMap v, int K, int D, CorrOut corr) {
  const long long total = (long long)K * (v.ld >> 2);
  const int blocks = (int)((total + 255) / 256 < 148LL * 16 ? (total + 255) / 256 : 148LL * 16);
  diff_rows_kernel<<<blocks, 256, 0, s>>>(Xa, Xb, v, K, D, corr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_cast_bf16(cudaStream_t s, const float* W, __nv_bfloat16* Wb, long long n) {
  const long long n4 = n / 4;   // J*D is a multiple of 4 on the bf16 path (D % 8 == 0 is required there)
  const int blocks = (int)((n4 + 255) / 256 < 148LL * 16 ? (n4 + 255) / 256 : 148LL * 16);
  cast_bf16_kernel<<<blocks, 256, 0, s>>>(W, Wb, n4);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

}  // namespace sfb
