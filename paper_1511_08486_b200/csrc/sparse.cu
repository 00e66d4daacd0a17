// Sparse-code paths of the sparse-coding dictionary update (Section 2, "Sparse coding"; Figure 3):
//
//   forward:  u_i = W a_i - x_i = sum_{(d,a) in code i} a * W[:, d] - x_i     (a_i given as a CSR row)
//   apply  :  W[:, d] -= eta * sum_{i : a_id != 0} a_id * u_i                 (only touched atoms move)
//
// W is J x D row-major, so an atom (column d) is strided in memory.  The forward therefore works on
// an atom-major copy W^T (one coalesced J-vector per nonzero), rebuilt from W by a tiled transpose.
// The apply gives every thread block a slab of 16 consecutive atoms (64 bytes of each of 1024 rows of
// W) held in shared memory; the block walks all samples in order, finds each sample's
// nonzeros inside its slab by binary search in the sorted CSR row, and applies them in (sample, atom)
// order.
// No floating-point atomics: every element of W is owned by one block and updated in a fixed order,
// so the result is bit-reproducible; atoms no code uses are written back unchanged.
#include "common.cuh"

namespace sfb {
namespace {

struct CsrRow {
  const uint32_t* idx;
  const float* val;
  int len;
};

__device__ __forceinline__ CsrRow csr_row(const CsrView& c, int i) {
  CsrRow r;
  if (c.base == nullptr) {
    uint32_t s = c.rowptr[i], e = c.rowptr[i + 1];
    if (c.cap_p > 0) {   // what the worker's stream can hold: the same truncation as pack_csr
      const uint32_t lim = c.rowptr[(size_t)(i / c.B) * c.B] + (uint32_t)c.cap_p;
      s = min(s, lim); e = min(e, lim);
    }
    r.idx = c.idx + s;
    r.val = c.val + s;
    r.len = (int)(e - s);
  } else {
    const int p = i / c.B, l = i % c.B;
    const char* vb = c.base + c.streams_off + (long long)p * c.stream_stride + c.v_off;
    const uint32_t* rp = reinterpret_cast<const uint32_t*>(vb);
    const uint32_t s = rp[l], e = rp[l + 1];
    r.idx = reinterpret_cast<const uint32_t*>(vb + c.rp_bytes) + s;
    r.val = reinterpret_cast<const float*>(vb + c.rp_bytes + c.idx_bytes) + s;
    r.len = (int)(e - s);
  }
  return r;
}

// Wt[d][j] = W[j][d]; Wt rows have ldt values (J rounded up to 4), pad columns zero.
__global__ void __launch_bounds__(256) transpose_kernel(const float* __restrict__ W, float* __restrict__ Wt, int J, int D,
                                                        int ldt) {
  __shared__ float tile[32][33];
  const int d0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
#pragma unroll
  for (int r = 0; r < 32; r += 8) {
    const int j = j0 + ty + r, d = d0 + tx;
    tile[ty + r][tx] = (j < J && d < D) ? W[(size_t)j * D + d] : 0.f;
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < 32; r += 8) {
    const int d = d0 + ty + r, j = j0 + tx;
    if (d < D && j < ldt) Wt[(size_t)d * ldt + j] = tile[tx][ty + r];
  }
}

// grid = (K samples, ceil(ldt / 1024)); each thread owns 4 consecutive rows j of W.
__global__ void __launch_bounds__(256) sc_forward_kernel(const float* __restrict__ Wt, int ldt, CsrView codes,
                                                         const float* __restrict__ Xdata, RowMap u, int K, int J, int D,
                                                         int* dev_status) {
  __shared__ uint32_t s_idx[256];
  __shared__ float s_val[256];
  const int i = blockIdx.x;
  const int j = (blockIdx.y * 256 + threadIdx.x) * 4;
  const CsrRow row = csr_row(codes, i);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int k0 = 0; k0 < row.len; k0 += 256) {
    const int k = k0 + threadIdx.x;
    uint32_t c = 0u;
    float a = 0.f;
    if (k < row.len) {
      c = row.idx[k];
      a = row.val[k];
      const bool bad = (c >= (uint32_t)D) || (k > 0 && row.idx[k - 1] >= c);
      if (bad) {
        if (blockIdx.y == 0) atomicOr(dev_status, SFB_DEV_BAD_INDEX);
        c = 0u;
        a = 0.f;   // the offending entry is skipped
      }
    }
    __syncthreads();
    s_idx[threadIdx.x] = c;
    s_val[threadIdx.x] = a;
    __syncthreads();
    const int n = min(256, row.len - k0);
    if (j < ldt) {
      // eight gathers in flight per thread before their multiply-adds (entries beyond n hold value 0, atom 0);
      // the order of the additions stays the order of the entries
      for (int e0 = 0; e0 < n; e0 += 8) {
        float4 w[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) w[q] = *reinterpret_cast<const float4*>(Wt + (size_t)s_idx[e0 + q] * ldt + j);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const float av = s_val[e0 + q];
          acc.x = fmaf(av, w[q].x, acc.x); acc.y = fmaf(av, w[q].y, acc.y);
          acc.z = fmaf(av, w[q].z, acc.z); acc.w = fmaf(av, w[q].w, acc.w);
        }
      }
    }
  }
  if (j < u.ld) {
    const float* x = Xdata + (size_t)i * J;
    float4 r;
    r.x = (j < J) ? acc.x - x[j] : 0.f;
    r.y = (j + 1 < J) ? acc.y - x[j + 1] : 0.f;
    r.z = (j + 2 < J) ? acc.z - x[j + 2] : 0.f;
    r.w = (j + 3 < J) ? acc.w - x[j + 3] : 0.f;
    *reinterpret_cast<float4*>(u.row(i) + (size_t)j * 4) = r;
  }
}

// One block per sample: zero the dense row, then scatter the sample's nonzeros into it.
__global__ void __launch_bounds__(256) densify_kernel(CsrView codes, RowMap a, int K, int D, int* dev_status,
                                                      bool round_tf32) {
  const int i = blockIdx.x;
  float* dst = reinterpret_cast<float*>(a.row(i));
  for (int q = threadIdx.x; q < (a.ld >> 2); q += 256) reinterpret_cast<float4*>(dst)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();
  const CsrRow row = csr_row(codes, i);
  for (int k = threadIdx.x; k < row.len; k += 256) {
    const uint32_t c = row.idx[k];
    if (c >= (uint32_t)D || (k > 0 && row.idx[k - 1] >= c)) atomicOr(dev_status, SFB_DEV_BAD_INDEX);   // entry skipped
    else {
      // the tensor cores drop the low 13 mantissa bits of a tf32 operand: rounding the code value to nearest
      // here (the dense rows are only ever a tf32 operand; the wire keeps the exact CSR values) halves that error
      uint32_t r = __float_as_uint(row.val[k]);
      if (round_tf32) asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(row.val[k]));
      dst[c] = __uint_as_float(r);
    }
  }
}

// The same through shared memory (one block per sample, the dense row of a.ld floats staged there), for the
// compensated path: the row goes out in whole 16-byte units together with its correction operands.
__global__ void __launch_bounds__(256) densify_corr_kernel(CsrView codes, RowMap a, int K, int D, int* dev_status,
                                                           CorrOut corr) {
  extern __shared__ __align__(16) float dense[];
  const int i = blockIdx.x;
  const int units = a.ld >> 2;
  for (int q = threadIdx.x; q < units; q += 256) reinterpret_cast<float4*>(dense)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();
  const CsrRow row = csr_row(codes, i);
  for (int k = threadIdx.x; k < row.len; k += 256) {
    const uint32_t c = row.idx[k];
    if (c >= (uint32_t)D || (k > 0 && row.idx[k - 1] >= c)) atomicOr(dev_status, SFB_DEV_BAD_INDEX);   // entry skipped
    else dense[c] = row.val[k];
  }
  __syncthreads();
  float4* dst = reinterpret_cast<float4*>(a.row(i));
  for (int q = threadIdx.x; q < units; q += 256) {
    const float4 t = reinterpret_cast<const float4*>(dense)[q];
    dst[q] = t;
    corr_store4(corr, i, a.B, q * 4, t);
  }
}

__global__ void __launch_bounds__(256) finish_sc_kernel(RowMap zr, RowMap u, const float* __restrict__ Xdata, int K, int J,
                                                        int nsplit, long long zstride, CorrOut corr) {
  const int units = u.ld >> 2;
  const long long total = (long long)K * units;
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < total;
       g += (long long)gridDim.x * blockDim.x) {
    const int i = (int)(g / units), j = (int)(g % units) * 4;
    float4* p = reinterpret_cast<float4*>(u.row(i) + (size_t)j * 4);
    const float* zp = reinterpret_cast<const float*>(zr.row(i)) + j;
    float4 z = *reinterpret_cast<const float4*>(zp);
    for (int sp = 1; sp < nsplit; ++sp) {
      const float4 q = *reinterpret_cast<const float4*>(zp + sp * zstride);
      z.x += q.x; z.y += q.y; z.z += q.z; z.w += q.w;
    }
    const float* x = Xdata + (size_t)i * J;
    z.x = (j < J) ? z.x - x[j] : 0.f;
    z.y = (j + 1 < J) ? z.y - x[j + 1] : 0.f;
    z.z = (j + 2 < J) ? z.z - x[j + 2] : 0.f;
    z.w = (j + 3 < J) ? z.w - x[j + 3] : 0.f;
    *p = z;
    if (corr.mn != nullptr) corr_store4(corr, i, u.B, j, z);
  }
}

constexpr int SLAB_D = 16;         // atoms per block: two 32-byte sectors of every row of W
constexpr int SLAB_T = 256;        // threads per block
constexpr int SLAB_J = 4 * SLAB_T; // rows of W per block: four consecutive rows per thread
constexpr int SLAB_CAP = 1024;     // entries applied per pass (more are handled by further passes)
constexpr int SLAB_BATCH = 8;      // entries whose u values are fetched together

// grid = (ceil(D / 16), ceil(J / 1024)); the block owns the 16-atom x 1024-row slab of W in shared memory.
// Per round of 256 samples: every thread finds the entries of one sample's sorted CSR row that fall
// inside the slab (binary search + short scan), a block-wide scan orders them by (sample, atom), and
// the entries are applied in that order: thread t adds -eta * a * u_i[j] to its own four rows j of
// the slab, with the u values of 8 entries fetched ahead as independent 16-byte loads.
// A thread owns its rows for the whole kernel, so there is no race and the summation order is fixed.
__global__ void __launch_bounds__(SLAB_T) sc_apply_kernel(float* __restrict__ W, CsrView codes, RowMap u, int K, int J,
                                                          int D, float eta, const int* __restrict__ status_ro) {
  extern __shared__ __align__(16) float Ws[];   // 64 KB: Ws[atom * SLAB_J + row]
  __shared__ int s_key[SLAB_CAP];               // sample * 16 + atom-in-slab
  __shared__ float s_val[SLAB_CAP];             // -eta * code value
  __shared__ int s_warp[SLAB_T / 32];
  if (status_ro != nullptr && (*status_ro & SFB_DEV_BAD_HEADER)) return;
  const int t = threadIdx.x;
  const int d0 = blockIdx.x * SLAB_D, j0 = blockIdx.y * SLAB_J;
  const int dn = min(SLAB_D, D - d0);
  const int jn = min(SLAB_J, J - j0);
  const bool vec_ok = ((D & 3) == 0) && (dn == SLAB_D);

  // slab in: thread handles whole rows (16 atoms = 64 bytes), transposed into Ws[atom][row]
  for (int jj = t; jj < SLAB_J; jj += SLAB_T) {
    float w[SLAB_D];
#pragma unroll
    for (int e = 0; e < SLAB_D; ++e) w[e] = 0.f;
    if (jj < jn) {
      const float* src = W + (size_t)(j0 + jj) * D + d0;
      if (vec_ok) {
#pragma unroll
        for (int q = 0; q < SLAB_D / 4; ++q) {
          const float4 v = *reinterpret_cast<const float4*>(src + 4 * q);
          w[4 * q] = v.x; w[4 * q + 1] = v.y; w[4 * q + 2] = v.z; w[4 * q + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int e = 0; e < SLAB_D; ++e)
          if (e < dn) w[e] = src[e];
      }
    }
#pragma unroll
    for (int e = 0; e < SLAB_D; ++e) Ws[e * SLAB_J + jj] = w[e];
  }
  __syncthreads();

  const int jt = 4 * t;                      // this thread's first row inside the slab
  const bool row_ok = jt < jn;               // J is padded to 4 in U rows, so a float4 never leaves the row
  for (int c0 = 0; c0 < K; c0 += SLAB_T) {
    // (1) this thread's sample: entries of its sorted row inside [d0, d0 + dn)
    const int i = c0 + t;
    int lo = 0, cnt = 0;
    CsrRow row;
    row.len = 0;
    if (i < K) {
      row = csr_row(codes, i);
      int hi = row.len;
      while (lo < hi) {   // lower bound of d0
        const int mid = (lo + hi) >> 1;
        if (row.idx[mid] < (uint32_t)d0) lo = mid + 1; else hi = mid;
      }
      // (the lower bound matters only for rows that are not ascending: nothing outside the slab is ever addressed)
      while (lo + cnt < row.len && cnt < SLAB_D && row.idx[lo + cnt] >= (uint32_t)d0 &&
             row.idx[lo + cnt] < (uint32_t)(d0 + dn))
        ++cnt;
    }
    // (2) block-wide exclusive scan of the counts (fixed order)
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if ((t & 31) >= o) incl += n;
    }
    if ((t & 31) == 31) s_warp[t >> 5] = incl;
    __syncthreads();
    if (t < 32) {
      int v = (t < SLAB_T / 32) ? s_warp[t] : 0;
#pragma unroll
      for (int o = 1; o < SLAB_T / 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, v, o);
        if (t >= o) v += n;
      }
      if (t < SLAB_T / 32) s_warp[t] = v;
    }
    __syncthreads();
    const int base = incl - cnt + ((t >> 5) > 0 ? s_warp[(t >> 5) - 1] : 0);
    const int total = s_warp[SLAB_T / 32 - 1];
    __syncthreads();
    // (3) apply, SLAB_CAP entries per pass, in (sample, atom) order
    for (int win = 0; win < total; win += SLAB_CAP) {
      for (int e = 0; e < cnt; ++e) {
        const int pos = base + e - win;
        if (pos >= 0 && pos < SLAB_CAP) {
          s_key[pos] = i * SLAB_D + ((int)row.idx[lo + e] - d0);
          // an entry that breaks the ascending order is skipped, as in the forward pass
          const bool skip = lo + e > 0 && row.idx[lo + e - 1] >= row.idx[lo + e];
          s_val[pos] = skip ? 0.f : -eta * row.val[lo + e];
        }
      }
      __syncthreads();
      const int n = min(SLAB_CAP, total - win);
      if (row_ok) {
        const char* ucol = u.base + (size_t)(j0 + jt) * 4;   // this thread's four columns of U
        for (int e0 = 0; e0 < n; e0 += SLAB_BATCH) {
          float4 uv[SLAB_BATCH];
#pragma unroll
          for (int q = 0; q < SLAB_BATCH; ++q) {   // independent loads first; repeats of one sample hit L1
            uv[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (e0 + q < n) {
              const int smp = s_key[e0 + q] / SLAB_D;
              uv[q] = __ldg(reinterpret_cast<const float4*>(ucol + (long long)(smp / u.B) * u.worker_stride +
                                                            (long long)(smp % u.B) * u.ld * 4));
            }
          }
#pragma unroll
          for (int q = 0; q < SLAB_BATCH; ++q) {
            if (e0 + q < n) {
              const float ca = s_val[e0 + q];
              float4* ws = reinterpret_cast<float4*>(Ws + (s_key[e0 + q] % SLAB_D) * SLAB_J + jt);
              float4 w = *ws;
              w.x = fmaf(ca, uv[q].x, w.x); w.y = fmaf(ca, uv[q].y, w.y);
              w.z = fmaf(ca, uv[q].z, w.z); w.w = fmaf(ca, uv[q].w, w.w);
              *ws = w;
            }
          }
        }
      }
      __syncthreads();
    }
  }

  for (int jj = t; jj < jn; jj += SLAB_T) {
    float* dst = W + (size_t)(j0 + jj) * D + d0;
    if (vec_ok) {
#pragma unroll
      for (int q = 0; q < SLAB_D / 4; ++q)
        *reinterpret_cast<float4*>(dst + 4 * q) =
            make_float4(Ws[(4 * q) * SLAB_J + jj], Ws[(4 * q + 1) * SLAB_J + jj], Ws[(4 * q + 2) * SLAB_J + jj],
                        Ws[(4 * q + 3) * SLAB_J + jj]);
    } else {
      for (int e = 0; e < dn; ++e) dst[e] = Ws[e * SLAB_J + jj];
    }
  }
}

}  // namespace

// Workspace the forward needs: the atom-major copy, D rows of ldt = roundup(J, 4) floats.
long long sc_forward_workspace_bytes(int J, int D) { return (long long)D * pad_to(J, 4) * 4; }

int launch_sc_forward_ws(cudaStream_t s, const float* W, float* Wt, CsrView codes, const float* Xdata, RowMap u, int K,
                         int J, int D, int* dev_status) {
  const int ldt = (int)pad_to(J, 4);
  dim3 tg((D + 31) / 32, (ldt + 31) / 32);
  transpose_kernel<<<tg, 256, 0, s>>>(W, Wt, J, D, ldt);
  const int cols = ldt > u.ld ? ldt : u.ld;   // pad columns of a wider u row are written (as zeros) too
  dim3 grid(K, (cols + 1023) / 1024);
  sc_forward_kernel<<<grid, 256, 0, s>>>(Wt, ldt, codes, Xdata, u, K, J, D, dev_status);
  return cudaGetLastError() == cudaSuccess ? 2 : SFB_ERR_CUDA;
}

int launch_densify_codes(cudaStream_t s, CsrView codes, RowMap a, int K, int D, int* dev_status, bool round_tf32) {
  densify_kernel<<<K, 256, 0, s>>>(codes, a, K, D, dev_status, round_tf32);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

bool densify_corr_fits(int ld) { return (size_t)ld * 4 <= 200 * 1024; }

int launch_densify_codes_corr(cudaStream_t s, CsrView codes, RowMap a, int K, int D, int* dev_status, CorrOut corr) {
  const size_t smem = (size_t)a.ld * 4;
  static PerDeviceOnce attr_once;   // function attributes are per device
  if (attr_once.first())
    cudaFuncSetAttribute(densify_corr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  densify_corr_kernel<<<K, 256, smem, s>>>(codes, a, K, D, dev_status, corr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_finish_sc(cudaStream_t s, RowMap z, RowMap u, const float* Xdata, int K, int J, int nsplit,
                     long long split_stride_bytes, CorrOut corr) {
  const long long total = (long long)K * (u.ld >> 2);
  const int blocks = (int)((total + 255) / 256 < 148LL * 16 ? (total + 255) / 256 : 148LL * 16);
  finish_sc_kernel<<<blocks, 256, 0, s>>>(z, u, Xdata, K, J, nsplit, split_stride_bytes / 4, corr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_sc_apply(cudaStream_t s, float* W, CsrView codes, RowMap u, int K, int J, int D, float eta,
                    const int* dev_status_ro, int* /*dev_status*/) {
  static PerDeviceOnce attr_once;   // function attributes are per device
  if (attr_once.first()) {
    cudaFuncSetAttribute(sc_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SLAB_D * SLAB_J * 4);
    cudaFuncSetAttribute(sc_apply_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
  }
  dim3 grid((D + SLAB_D - 1) / SLAB_D, (J + SLAB_J - 1) / SLAB_J);
  sc_apply_kernel<<<grid, SLAB_T, SLAB_D * SLAB_J * 4, s>>>(W, codes, u, K, J, D, eta, dev_status_ro);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

}  // namespace sfb
