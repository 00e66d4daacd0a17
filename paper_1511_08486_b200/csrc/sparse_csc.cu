// Sparse-v scatter apply through an atom-major (CSC) view of the codes.
//
//   W[:, d] -= eta * sum_{i : a_id != 0} a_id * u_i        (Section 3 update with v_i = a_i sparse)
//
// The codes arrive sample-major (CSR, the factor v_i of each sample).  Per step they are re-sorted by
// atom with a counting sort that is deterministic: counts per (chunk of 8 samples, atom) by integer
// atomics, prefix sums over chunks and atoms, then every chunk places its samples one after the other,
// so inside a column the entries are in sample order whatever the thread schedule.
// The apply gives each thread block 32 rows of W and keeps the matching 32 columns of ALL u_i in shared
// memory (K x 128 bytes).  A warp takes 32 consecutive atoms: for each atom it walks the column's
// entries (coalesced loads, broadcast by shuffles), accumulating a_id * u_i[j0 + lane] from shared
// memory, parks the 32 sums in a private 32 x 33 tile, and finally updates W with 128-byte row segments.
// W and U are each read once; no floating-point atomics; every element of W has one owner and a fixed
// summation order (bit-reproducible); atoms nobody uses get W + (-eta * 0) = W, bit-identical.
#include "common.cuh"

namespace sfb {
namespace {

constexpr int CSC_CHUNK = 8;    // samples per chunk of the counting sort
constexpr int CSC_JT = 32;      // rows of W per block of the apply

struct CsrRow2 {
  const uint32_t* idx;
  const float* val;
  int len;
};
__device__ __forceinline__ CsrRow2 csr_row2(const CsrView& c, int i) {
  CsrRow2 r;
  if (c.base == nullptr) {
    const uint32_t s = c.rowptr[i], e = c.rowptr[i + 1];
    r.idx = c.idx + s; r.val = c.val + s; r.len = (int)(e - s);
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

// cnt[chunk][d] += 1 for every nonzero (integer atomics: the final counts do not depend on the order)
__global__ void __launch_bounds__(256) csc_count_kernel(CsrView codes, int K, int D, int* __restrict__ cnt) {
  const int i = blockIdx.x;
  const CsrRow2 row = csr_row2(codes, i);
  int* c = cnt + (size_t)(i / CSC_CHUNK) * D;
  for (int k = threadIdx.x; k < row.len; k += 256) {
    const uint32_t d = row.idx[k];
    if (d < (uint32_t)D) atomicAdd(c + d, 1);
  }
}

// per atom: counts per chunk -> offsets of each chunk inside the column; column totals
__global__ void __launch_bounds__(256) csc_chunk_offsets_kernel(int nchunks, int D, int* __restrict__ cnt,
                                                                int* __restrict__ total) {
  const int d = blockIdx.x * 256 + threadIdx.x;
  if (d >= D) return;
  int run = 0;
  for (int c0 = 0; c0 < nchunks; c0 += 8) {   // eight independent loads in flight, then the running sum
    int t[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) t[q] = (c0 + q < nchunks) ? cnt[(size_t)(c0 + q) * D + d] : 0;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (c0 + q < nchunks) cnt[(size_t)(c0 + q) * D + d] = run;
      run += t[q];
    }
  }
  total[d] = run;
}

// colptr = exclusive scan of total (one block, fixed order)
__global__ void __launch_bounds__(1024) csc_scan_kernel(int D, const int* __restrict__ total, int* __restrict__ colptr) {
  __shared__ int warp_sum[32];
  __shared__ int carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < D; base += 1024) {
    const int d = base + threadIdx.x;
    const int v = d < D ? total[d] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if ((threadIdx.x & 31) >= o) incl += n;
    }
    if ((threadIdx.x & 31) == 31) warp_sum[threadIdx.x >> 5] = incl;
    __syncthreads();
    if (threadIdx.x < 32) {
      int w = warp_sum[threadIdx.x];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, w, o);
        if (threadIdx.x >= o) w += n;
      }
      warp_sum[threadIdx.x] = w;
    }
    __syncthreads();
    const int before = carry + ((threadIdx.x >> 5) > 0 ? warp_sum[(threadIdx.x >> 5) - 1] : 0) + incl - v;
    if (d < D) colptr[d] = before;
    __syncthreads();
    if (threadIdx.x == 1023) carry = before + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) colptr[D] = carry;
}

// one block per chunk: its samples are placed one after the other, so a column is in sample order
__global__ void __launch_bounds__(256) csc_fill_kernel(CsrView codes, int K, int D, int* __restrict__ cnt,
                                                       const int* __restrict__ colptr, int* __restrict__ ent_i,
                                                       float* __restrict__ ent_a) {
  const int c = blockIdx.x;
  int* off = cnt + (size_t)c * D;
  for (int s = 0; s < CSC_CHUNK; ++s) {
    const int i = c * CSC_CHUNK + s;
    if (i < K) {
      const CsrRow2 row = csr_row2(codes, i);
      for (int k = threadIdx.x; k < row.len; k += 256) {
        const uint32_t d = row.idx[k];
        if (d < (uint32_t)D) {      // indices are unique inside a row: one writer per (chunk, atom) per step
          const int pos = colptr[d] + off[d];
          off[d] += 1;
          ent_i[pos] = i;
          ent_a[pos] = row.val[k];
        }
      }
    }
    __syncthreads();
  }
}

// grid = ceil(J / 32); dynamic shared memory: K * 32 floats (u columns) + warps * 32 * 33 floats (tiles)
__global__ void __launch_bounds__(512) csc_apply_kernel(float* __restrict__ W, RowMap u, int K, int J, int D, float eta,
                                                        const int* __restrict__ colptr, const int* __restrict__ ent_i,
                                                        const float* __restrict__ ent_a,
                                                        const int* __restrict__ status_ro) {
  extern __shared__ __align__(16) float smem[];
  if (status_ro != nullptr && (*status_ro & SFB_DEV_BAD_HEADER)) return;
  float* Us = smem;                                   // [K][32]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  float* T = smem + (size_t)K * 32 + warp * (32 * 33 + 64);   // [32][33] + entry strip, private to the warp
  const int j0 = blockIdx.x * CSC_JT;
  const bool jok = j0 + lane < J;
  for (int i = warp; i < K; i += nwarps)
    Us[i * 32 + lane] = jok ? reinterpret_cast<const float*>(u.row(i))[j0 + lane] : 0.f;
  __syncthreads();

  const int nblocks = (D + 31) / 32;
  for (int ab = warp; ab < nblocks; ab += nwarps) {
    const int d0 = ab * 32;
    const int dn = min(32, D - d0);
    // column boundaries of the 32 atoms: lane holds colptr[d0 + lane] and the end of the last one
    const int cp = colptr[min(d0 + lane, D)];
    const int cp_next = colptr[min(d0 + 32, D)];
    // per atom: rounds of 32 entries staged in a per-warp shared-memory strip (one coalesced load per
    // round, the next round's load already in flight), then one broadcast read + one u read + one FMA
    // per entry, four running sums
    int2* strip = reinterpret_cast<int2*>(T + 32 * 33);           // 32 (sample, value) pairs
    int pre_i = 0;
    float pre_a = 0.f;
    {
      const int b0 = __shfl_sync(0xffffffffu, cp, 0);
      if (b0 + lane < cp_next) { pre_i = ent_i[b0 + lane]; pre_a = ent_a[b0 + lane]; }
    }
    for (int dd = 0; dd < dn; ++dd) {
      const int beg = __shfl_sync(0xffffffffu, cp, dd);
      const int stop = (dd < 31) ? __shfl_sync(0xffffffffu, cp, dd + 1) : cp_next;
      float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
      for (int base = beg; base < stop; base += 32) {
        // the prefetched values are those of [base, base + 32) of the contiguous entry range
        strip[lane] = make_int2(base + lane < stop ? pre_i : 0, __float_as_int(base + lane < stop ? pre_a : 0.f));
        const int nxt = (base + 32 < stop) ? base + 32 : stop;    // next round: same atom, or the next atom's start
        if (nxt + lane < cp_next) { pre_i = ent_i[nxt + lane]; pre_a = ent_a[nxt + lane]; }
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 32; k += 4) {
          const int2 e0 = strip[k], e1 = strip[k + 1], e2 = strip[k + 2], e3 = strip[k + 3];
          acc0 = fmaf(__int_as_float(e0.y), Us[e0.x * 32 + lane], acc0);
          acc1 = fmaf(__int_as_float(e1.y), Us[e1.x * 32 + lane], acc1);
          acc2 = fmaf(__int_as_float(e2.y), Us[e2.x * 32 + lane], acc2);
          acc3 = fmaf(__int_as_float(e3.y), Us[e3.x * 32 + lane], acc3);
        }
        __syncwarp();
      }
      T[dd * 33 + lane] = (acc0 + acc1) + (acc2 + acc3);
    }
    __syncwarp();
    // W[j0 + jj][d0 + lane] -= eta * T[lane][jj]: 128-byte row segments, 8 rows fetched at a time
    if (lane < dn) {
      const int jn = min(32, J - j0);
      for (int jb = 0; jb < jn; jb += 8) {
        float wv[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
          wv[q] = (jb + q < jn) ? W[(size_t)(j0 + jb + q) * D + d0 + lane] : 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (jb + q < jn) W[(size_t)(j0 + jb + q) * D + d0 + lane] = fmaf(-eta, T[lane * 33 + jb + q], wv[q]);
      }
    }
    __syncwarp();
  }
}

}  // namespace

// Scratch of the CSC path: counts [nchunks][D] + totals [D] + colptr [D + 1] ints, entries (int + float) x nnz_capacity.
long long sc_csc_workspace_bytes(int K, int D, long long nnz_capacity) {
  const long long nchunks = (K + CSC_CHUNK - 1) / CSC_CHUNK;
  return pad_to((nchunks * D + D + D + 1) * 4, 256) + pad_to(nnz_capacity * 4, 256) * 2;
}

// The u columns of all K samples must fit in shared memory next to the warps' tiles.
bool sc_csc_supported(int K) { return (long long)K * 128 + 16 * (32 * 33 + 64) * 4 <= 220 * 1024; }

int launch_sc_apply_csc(cudaStream_t s, float* W, CsrView codes, RowMap u, int K, int J, int D, float eta,
                        long long nnz_capacity, void* workspace, const int* dev_status_ro) {
  const int nchunks = (K + CSC_CHUNK - 1) / CSC_CHUNK;
  int* cnt = reinterpret_cast<int*>(workspace);
  int* total = cnt + (size_t)nchunks * D;
  int* colptr = total + D;
  char* ent_base = reinterpret_cast<char*>(workspace) + pad_to(((long long)nchunks * D + D + D + 1) * 4, 256);
  int* ent_i = reinterpret_cast<int*>(ent_base);
  float* ent_a = reinterpret_cast<float*>(ent_base + pad_to(nnz_capacity * 4, 256));
  if (cudaMemsetAsync(cnt, 0, (size_t)nchunks * D * 4, s) != cudaSuccess) return SFB_ERR_CUDA;
  csc_count_kernel<<<K, 256, 0, s>>>(codes, K, D, cnt);
  csc_chunk_offsets_kernel<<<(D + 255) / 256, 256, 0, s>>>(nchunks, D, cnt, total);
  csc_scan_kernel<<<1, 1024, 0, s>>>(D, total, colptr);
  csc_fill_kernel<<<nchunks, 256, 0, s>>>(codes, K, D, cnt, colptr, ent_i, ent_a);
  const int threads = 512;
  const size_t smem = (size_t)K * 128 + (size_t)(threads / 32) * (32 * 33 + 64) * 4;
  static bool attr_done = false;
  if (!attr_done) {
    cudaFuncSetAttribute(csc_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
    attr_done = true;
  }
  csc_apply_kernel<<<(J + CSC_JT - 1) / CSC_JT, threads, smem, s>>>(W, u, K, J, D, eta, colptr, ent_i, ent_a,
                                                                  dev_status_ro);
  return cudaGetLastError() == cudaSuccess ? 5 : SFB_ERR_CUDA;
}

}  // namespace sfb
