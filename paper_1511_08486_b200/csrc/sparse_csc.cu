// Sparse-v scatter apply through an atom-major (CSC) view of the codes.
//
//   W[:, d] -= eta * sum_{i : a_id != 0} a_id * u_i        (Section 3 update with v_i = a_i sparse)
//
// The codes arrive sample-major (CSR, the factor v_i of each sample).  Per step they are re-sorted by
// atom with a counting sort that is deterministic: counts per (chunk of 8 samples, atom) by integer
// atomics, prefix sums over chunks and atoms, then every chunk places its samples one after the other,
// so inside a column the entries are in sample order whatever the thread schedule.
// The apply gives each thread block 64 rows of W and keeps the matching 64 columns of a slice of the
// u_i in shared memory (the samples are taken in as few slices as fit).  A warp takes 16 consecutive
// atoms: for each atom it walks the slice's entries of the column (coalesced loads staged through a
// small per-warp strip), accumulating a_id * u_i[j0 + 2 lane .. + 1] from shared memory, parks the sums
// in a private 16 x 65 tile, and finally updates W with 64-byte row segments.
// U is read once and W once per slice; no floating-point atomics; every element of W has one owner and a fixed
// summation order (bit-reproducible); atoms nobody uses get W + (-eta * 0) = W, bit-identical.
#include <type_traits>

#include "common.cuh"

namespace sfb {
namespace {

constexpr int CSC_CHUNK = 8;    // samples per chunk of the counting sort

struct CsrRow2 {
  const uint32_t* idx;
  const float* val;
  int len;
};
__device__ __forceinline__ CsrRow2 csr_row2(const CsrView& c, int i) {
  CsrRow2 r;
  if (c.base == nullptr) {
    uint32_t s = c.rowptr[i], e = c.rowptr[i + 1];
    if (c.cap_p > 0) {   // what the worker's stream can hold: the same truncation as pack_csr
      const uint32_t lim = c.rowptr[(size_t)(i / c.B) * c.B] + (uint32_t)c.cap_p;
      s = min(s, lim); e = min(e, lim);
    }
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

// An entry counts only if its atom exists and the row is strictly ascending up to it: the rule of the forward
// pass (sc_forward_kernel), so that forward and apply agree on malformed rows, and the reason why a
// (chunk, atom) cell has at most one writer per sample in the fill below (no repeated atom inside a row).
__device__ __forceinline__ bool entry_ok(const CsrRow2& row, int k, int D) {
  const uint32_t d = row.idx[k];
  return d < (uint32_t)D && !(k > 0 && row.idx[k - 1] >= d);
}

// cnt[chunk][d] += 1 for every nonzero (integer atomics: the final counts do not depend on the order)
__global__ void __launch_bounds__(256) csc_count_kernel(CsrView codes, int K, int D, int* __restrict__ cnt,
                                                        int* dev_status) {
  const int i = blockIdx.x;
  const CsrRow2 row = csr_row2(codes, i);
  int* c = cnt + (size_t)(i / CSC_CHUNK) * D;
  bool bad = false;
  for (int k = threadIdx.x; k < row.len; k += 256) {
    if (entry_ok(row, k, D)) atomicAdd(c + row.idx[k], 1);
    else bad = true;   // the entry is skipped
  }
  if (bad && dev_status != nullptr) atomicOr(dev_status, SFB_DEV_BAD_INDEX);
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
        if (entry_ok(row, k, D)) {  // indices that pass are unique inside a row: one writer per (chunk, atom) per step
          const uint32_t d = row.idx[k];
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

constexpr int CSC2_JT = 64;     // rows of W per block of the two-rows-per-lane apply
constexpr int CSC2_AB = 16;     // atoms per warp block there
constexpr int CSC2_WARP_FLOATS = 64 + CSC2_AB * 65;   // entry strip (32 x 8 bytes) + [16][65] tile

// Two rows of W per lane, the samples taken in `passes` slices so that a slice of the u columns
// (Kh x 256 bytes) fits in shared memory.  Shared-memory bandwidth bounds this kernel: per entry and 64 rows
// it costs half a broadcast read of the strip (two entries per 16-byte load) and one 256-byte read of u.
// grid = (ceil(J / 64), atom splits).  cnt holds, after the fill, for every (chunk, atom) the number of
// entries of the column that belong to samples before the END of the chunk, which gives the slice bounds.
__global__ void __launch_bounds__(512) csc_apply_kernel(float* __restrict__ W, RowMap u, int K, int J, int D, float eta,
                                                         const int* __restrict__ colptr, const int* __restrict__ cnt,
                                                         const int* __restrict__ ent_i, const float* __restrict__ ent_a,
                                                         int passes, int Kh, const int* __restrict__ status_ro) {
  extern __shared__ __align__(16) float smem[];
  if (status_ro != nullptr && (*status_ro & SFB_DEV_BAD_HEADER)) return;
  float* Us = smem;                                   // [Kh][64]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  float* region = smem + (size_t)Kh * 64 + warp * CSC2_WARP_FLOATS;
  int2* strip = reinterpret_cast<int2*>(region);
  const int4* strip4 = reinterpret_cast<const int4*>(region);
  float* T = region + 64;
  const int j0 = blockIdx.x * CSC2_JT;
  const int jn = min(CSC2_JT, J - j0);
  const int nnz = colptr[D];
  const int nchunks = (K + CSC_CHUNK - 1) / CSC_CHUNK;
  const int nblocks = (D + CSC2_AB - 1) / CSC2_AB;
  for (int h = 0; h < passes; ++h) {
    const int i_lo = h * Kh;
    if (i_lo >= K) break;
    const int i_n = min(Kh, K - i_lo);
    __syncthreads();                                  // the previous slice is no longer read
    for (int i = warp; i < i_n; i += nwarps) {
      const float* ur = reinterpret_cast<const float*>(u.row(i_lo + i)) + j0;
      float2 v = make_float2(0.f, 0.f);
      if (2 * lane + 1 < jn) v = *reinterpret_cast<const float2*>(ur + 2 * lane);
      else if (2 * lane < jn) v.x = ur[2 * lane];
      *reinterpret_cast<float2*>(Us + i * 64 + 2 * lane) = v;
    }
    __syncthreads();
    const int c_lo = i_lo / CSC_CHUNK;                               // Kh is a multiple of the chunk size
    const int c_hi = min(nchunks, (i_lo + Kh) / CSC_CHUNK);
    for (int ab = blockIdx.y + gridDim.y * warp; ab < nblocks; ab += gridDim.y * nwarps) {
      const int d0 = ab * CSC2_AB;
      const int dn = min(CSC2_AB, D - d0);
      int lo = nnz, hi = nnz;                                        // entry range of atom d0 + lane in this slice
      if (lane < dn) {
        const int d = d0 + lane, cp = colptr[d];
        lo = (c_lo == 0) ? cp : cp + cnt[(size_t)(c_lo - 1) * D + d];
        hi = cp + cnt[(size_t)(c_hi - 1) * D + d];
      }
      int pre_i = 0;
      float pre_a = 0.f;
      {
        const int b0 = __shfl_sync(0xffffffffu, lo, 0);
        if (b0 + lane < nnz) { pre_i = ent_i[b0 + lane]; pre_a = ent_a[b0 + lane]; }
      }
      for (int dd = 0; dd < dn; ++dd) {
        const int beg = __shfl_sync(0xffffffffu, lo, dd);
        const int stop = __shfl_sync(0xffffffffu, hi, dd);
        const int next_beg = __shfl_sync(0xffffffffu, lo, dd + 1);   // lane 16 and up hold nnz: nothing to fetch
        float2 acc0 = make_float2(0.f, 0.f), acc1 = acc0, acc2 = acc0, acc3 = acc0;
        if (beg >= stop && next_beg + lane < nnz) { pre_i = ent_i[next_beg + lane]; pre_a = ent_a[next_beg + lane]; }
        for (int base = beg; base < stop; base += 32) {
          const bool ok = base + lane < stop;
          // the sample index addresses shared memory: keep it inside the slice whatever the entry arrays hold
          const int li = min(max(pre_i - i_lo, 0), i_n - 1);
          strip[lane] = make_int2(ok ? li : 0, __float_as_int(ok ? pre_a : 0.f));
          const int nxt = (base + 32 < stop) ? base + 32 : next_beg;
          if (nxt + lane < nnz) { pre_i = ent_i[nxt + lane]; pre_a = ent_a[nxt + lane]; }
          __syncwarp();
          // a round holds up to 32 entries; short columns (sparse codes) take the 8- or 16-entry body, so the time of
          // a column follows its entries, not the round size (the bodies are unrolled: no branch inside them)
          const int n_here = min(32, stop - base);     // warp-uniform
          auto body = [&](auto iters) {
#pragma unroll
            for (int k = 0; k < decltype(iters)::value; k += 2) {
              const int4 p = strip4[k], q = strip4[k + 1];
              const float2 u0 = *reinterpret_cast<const float2*>(Us + p.x * 64 + 2 * lane);
              const float2 u1 = *reinterpret_cast<const float2*>(Us + p.z * 64 + 2 * lane);
              const float2 u2 = *reinterpret_cast<const float2*>(Us + q.x * 64 + 2 * lane);
              const float2 u3 = *reinterpret_cast<const float2*>(Us + q.z * 64 + 2 * lane);
              acc0.x = fmaf(__int_as_float(p.y), u0.x, acc0.x); acc0.y = fmaf(__int_as_float(p.y), u0.y, acc0.y);
              acc1.x = fmaf(__int_as_float(p.w), u1.x, acc1.x); acc1.y = fmaf(__int_as_float(p.w), u1.y, acc1.y);
              acc2.x = fmaf(__int_as_float(q.y), u2.x, acc2.x); acc2.y = fmaf(__int_as_float(q.y), u2.y, acc2.y);
              acc3.x = fmaf(__int_as_float(q.w), u3.x, acc3.x); acc3.y = fmaf(__int_as_float(q.w), u3.y, acc3.y);
            }
          };
          if (n_here <= 8) body(std::integral_constant<int, 4>());
          else if (n_here <= 16) body(std::integral_constant<int, 8>());
          else body(std::integral_constant<int, 16>());
          __syncwarp();
        }
        T[dd * 65 + 2 * lane] = (acc0.x + acc1.x) + (acc2.x + acc3.x);
        T[dd * 65 + 2 * lane + 1] = (acc0.y + acc1.y) + (acc2.y + acc3.y);
      }
      __syncwarp();
      // W[j0 + jj][d0 + a] -= eta * T[a][jj]: a warp instruction covers two rows x 16 atoms (64-byte segments)
      const int a = lane & 15, q = lane >> 4;
      if (a < dn) {
        for (int jb = 0; jb < jn; jb += 16) {
          float wv[8];
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const int jj = jb + 2 * t + q;
            wv[t] = (jj < jn) ? W[(size_t)(j0 + jj) * D + d0 + a] : 0.f;
          }
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const int jj = jb + 2 * t + q;
            if (jj < jn) W[(size_t)(j0 + jj) * D + d0 + a] = fmaf(-eta, T[a * 65 + jj], wv[t]);
          }
        }
      }
      __syncwarp();
    }
  }
}

}  // namespace

// Scratch of the CSC path: counts [nchunks][D] + totals [D] + colptr [D + 1] ints, entries (int + float) x nnz_capacity.
long long sc_csc_workspace_bytes(int K, int D, long long nnz_capacity) {
  const long long nchunks = (K + CSC_CHUNK - 1) / CSC_CHUNK;
  return pad_to((nchunks * D + D + D + 1) * 4, 256) + pad_to(nnz_capacity * 4, 256) * 2;
}

// The sliced kernel takes any K (more slices); the bound only keeps the chunk tables small.
bool sc_csc_supported(int K) { return K <= (1 << 14); }

namespace {
struct CscScratch {
  int* cnt; int* total; int* colptr; int* ent_i; float* ent_a;
};
CscScratch csc_scratch(void* workspace, int K, int D, long long nnz_capacity) {
  const int nchunks = (K + CSC_CHUNK - 1) / CSC_CHUNK;
  CscScratch w;
  w.cnt = reinterpret_cast<int*>(workspace);
  w.total = w.cnt + (size_t)nchunks * D;
  w.colptr = w.total + D;
  char* ent_base = reinterpret_cast<char*>(workspace) + pad_to(((long long)nchunks * D + D + D + 1) * 4, 256);
  w.ent_i = reinterpret_cast<int*>(ent_base);
  w.ent_a = reinterpret_cast<float*>(ent_base + pad_to(nnz_capacity * 4, 256));
  return w;
}
}  // namespace

// Atom-major re-sort of the codes into the workspace.  Reads the codes only (not u), so it may run beside
// the forward pass that produces u.
int launch_sc_csc_build(cudaStream_t s, CsrView codes, int K, int D, long long nnz_capacity, void* workspace,
                        int* dev_status) {
  const int nchunks = (K + CSC_CHUNK - 1) / CSC_CHUNK;
  const CscScratch w = csc_scratch(workspace, K, D, nnz_capacity);
  if (cudaMemsetAsync(w.cnt, 0, (size_t)nchunks * D * 4, s) != cudaSuccess) return SFB_ERR_CUDA;
  csc_count_kernel<<<K, 256, 0, s>>>(codes, K, D, w.cnt, dev_status);
  csc_chunk_offsets_kernel<<<(D + 255) / 256, 256, 0, s>>>(nchunks, D, w.cnt, w.total);
  csc_scan_kernel<<<1, 1024, 0, s>>>(D, w.total, w.colptr);
  csc_fill_kernel<<<nchunks, 256, 0, s>>>(codes, K, D, w.cnt, w.colptr, w.ent_i, w.ent_a);
  return cudaGetLastError() == cudaSuccess ? 4 : SFB_ERR_CUDA;
}

// The update from a workspace that launch_sc_csc_build filled for the same K, D and codes.
int launch_sc_csc_apply(cudaStream_t s, float* W, RowMap u, int K, int J, int D, float eta, long long nnz_capacity,
                        void* workspace, const int* dev_status_ro) {
  const CscScratch w = csc_scratch(workspace, K, D, nnz_capacity);
  const int threads = 512;
  static PerDeviceOnce attr_once;   // function attributes are per device
  if (attr_once.first())
    cudaFuncSetAttribute(csc_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
  // slices of the samples: the fewest that let Kh x 256 bytes of u sit beside the warps' tiles
  const long long tiles = (long long)(threads / 32) * CSC2_WARP_FLOATS * 4;
  const int kh_max = (int)((220 * 1024 - tiles) / 256) / CSC_CHUNK * CSC_CHUNK;
  const int passes = (K + kh_max - 1) / kh_max;
  const int Kh = ((K + passes - 1) / passes + CSC_CHUNK - 1) / CSC_CHUNK * CSC_CHUNK;
  const int nj = (J + CSC2_JT - 1) / CSC2_JT;
  const int nblocks = (D + CSC2_AB - 1) / CSC2_AB;
  int splits = 148 / nj;                            // atom splits: fill the SMs when J / 64 alone does not
  if (splits > nblocks / (threads / 32)) splits = nblocks / (threads / 32);
  if (splits < 1) splits = 1;
  const size_t smem = (size_t)Kh * 256 + (size_t)tiles;
  csc_apply_kernel<<<dim3(nj, splits), threads, smem, s>>>(W, u, K, J, D, eta, w.colptr, w.cnt, w.ent_i, w.ent_a, passes,
                                                          Kh, dev_status_ro);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_sc_apply_csc(cudaStream_t s, float* W, CsrView codes, RowMap u, int K, int J, int D, float eta,
                        long long nnz_capacity, void* workspace, const int* dev_status_ro) {
  const int a = launch_sc_csc_build(s, codes, K, D, nnz_capacity, workspace, const_cast<int*>(dev_status_ro));
  if (a < 0) return a;
  const int b2 = launch_sc_csc_apply(s, W, u, K, J, D, eta, nnz_capacity, workspace, dev_status_ro);
  return b2 < 0 ? b2 : a + b2;
}

}  // namespace sfb
