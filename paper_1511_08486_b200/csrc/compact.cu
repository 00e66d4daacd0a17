// Inactive-pair compaction of a committed SF buffer (dense v).
//
// A sufficient-factor pair whose u is all zeros (a dissimilar DML pair beyond the margin) contributes
// u v^T = 0 to the update, so a worker need not broadcast it (Section 6.1 of the paper: the sufficient
// factors are sparse and that is used; Section 5.1 counts the broadcast in pairs).  Per worker, the pairs
// with a nonzero u move to the front of the worker's B slots, in their original order, in both the U and the
// V block; the slots behind them are cleared; the directory gets the worker's own pair count and header flag
// bit 1 is set.  Offsets and strides of the buffer do not change.
//
// In place and deterministic: a row only ever moves to a lower slot of its own worker, and every block of the
// move kernel owns one (worker, 256-byte column slice) and walks the rows in waves of 64: a wave is read whole into
// shared memory before any of its rows is written, and the slots it writes were all read by then.
#include "common.cuh"

namespace sfb {
namespace {

constexpr int WAVE = 64;          // rows per wave of the move
constexpr int SLICE_UNITS = 16;   // 16-byte units per column slice (256 B): many small blocks hide the latency

// flags[i] = 1 if the wire values of u row i are not all zero (-0 counts as zero).  One warp per row.
__global__ void __launch_bounds__(256) row_nonzero_kernel(RowMap u, int K, int J, uint8_t* __restrict__ flags) {
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= K) return;
  const int per = 16 / u.es, units = (J + per - 1) / per;     // pad values inside the last unit are zeros
  const uint4* row = reinterpret_cast<const uint4*>(u.row(i));
  const uint32_t mask = u.es == 4 ? 0x7fffffffu : 0x7fff7fffu;
  uint32_t any = 0u;
  for (int q = lane; q < units; q += 32) {
    const uint4 w = row[q];
    any |= (w.x | w.y | w.z | w.w) & mask;
  }
  any = __any_sync(0xffffffffu, any != 0u) ? 1u : 0u;
  if (lane == 0) flags[i] = (uint8_t)any;
}

// One block per worker: dest[i] = new slot of pair i inside its worker (-1: left out); the worker's count goes
// to counts[p] and to the n_sf field of its directory entry; block 0 sets the header's "compacted" flag.
__global__ void __launch_bounds__(256) compact_scan_kernel(const uint8_t* __restrict__ flags, int B, int* __restrict__ dest,
                                                           int* __restrict__ counts, char* buf, int first_worker) {
  __shared__ int warp_cnt[8];
  __shared__ int base;
  const int p = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int start = 0; start < B; start += 256) {
    const int r = start + threadIdx.x;
    const bool f = r < B && flags[(size_t)p * B + r] != 0;
    const unsigned m = __ballot_sync(0xffffffffu, f);
    if (lane == 0) warp_cnt[warp] = __popc(m);
    __syncthreads();
    int off = base;
    for (int w = 0; w < warp; ++w) off += warp_cnt[w];
    if (r < B) dest[(size_t)p * B + r] = f ? off + __popc(m & ((1u << lane) - 1u)) : -1;
    __syncthreads();
    if (threadIdx.x == 0) {
      int t = 0;
      for (int w = 0; w < 8; ++w) t += warp_cnt[w];
      base += t;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    counts[p] = base;
    reinterpret_cast<uint32_t*>(buf + 128 + (size_t)(first_worker + p) * 32)[1] = (uint32_t)base;   // directory: n_sf
    if (p == 0) reinterpret_cast<uint32_t*>(buf)[2] |= 2u;                                            // header flags, bit 1
  }
}

// grid = (P, slices of the U rows + slices of the V rows).  Moves this block's 256-byte column slice of every kept
// row of worker p to its new slot and clears the slice in the slots behind the last kept row.
__global__ void __launch_bounds__(256) compact_move_kernel(char* streams, long long stream_stride, long long v_off, int B,
                                                           int u_units, int v_units, int u_slices,
                                                           const int* __restrict__ dest, const int* __restrict__ counts) {
  __shared__ uint4 wave[WAVE * SLICE_UNITS];   // 16 KB
  __shared__ int s_dest[WAVE];
  const int p = blockIdx.x;
  const bool is_v = (int)blockIdx.y >= u_slices;
  const int slice = is_v ? blockIdx.y - u_slices : blockIdx.y;
  const int row_units = is_v ? v_units : u_units;                 // 16-byte units per row
  const int q0 = slice * SLICE_UNITS;
  const int nq = min(SLICE_UNITS, row_units - q0);                // units of this slice that exist
  uint4* block = reinterpret_cast<uint4*>(streams + (size_t)p * stream_stride + (is_v ? v_off : 0));
  const int n_keep = counts[p];
  if (n_keep == B) return;                                        // nothing left out: every row stays where it is
  for (int r0 = 0; r0 < B; r0 += WAVE) {
    if (threadIdx.x < WAVE) s_dest[threadIdx.x] = (r0 + threadIdx.x < B) ? dest[(size_t)p * B + r0 + threadIdx.x] : -1;
    __syncthreads();
    for (int t = threadIdx.x; t < WAVE * SLICE_UNITS; t += 256) {
      const int r = t / SLICE_UNITS, q = t % SLICE_UNITS;
      if (q < nq && s_dest[r] >= 0 && s_dest[r] != r0 + r) wave[t] = block[(size_t)(r0 + r) * row_units + q0 + q];
    }
    __syncthreads();
    for (int t = threadIdx.x; t < WAVE * SLICE_UNITS; t += 256) {
      const int r = t / SLICE_UNITS, q = t % SLICE_UNITS;
      if (q < nq && s_dest[r] >= 0 && s_dest[r] != r0 + r) block[(size_t)s_dest[r] * row_units + q0 + q] = wave[t];
    }
    __syncthreads();
  }
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  const int tail = B - n_keep;
  for (int t = threadIdx.x; t < tail * nq; t += 256) {
    const int r = n_keep + t / nq, q = t % nq;
    block[(size_t)r * row_units + q0 + q] = zero;
  }
}

// idx[0 .. *n_out) = p * B + r for every worker p < workers and every r < its pair count, in that order.
__global__ void __launch_bounds__(256) kept_rows_kernel(const char* buf, int B, int workers, int* __restrict__ idx,
                                                        int* __restrict__ n_out) {
  __shared__ int base;
  if (threadIdx.x == 0) base = 0;
  __syncthreads();
  for (int p = 0; p < workers; ++p) {
    int n = (int)reinterpret_cast<const uint32_t*>(buf + 128 + (size_t)p * 32)[1];
    n = n < B ? n : B;
    const int b = base;
    for (int r = threadIdx.x; r < n; r += 256) idx[b + r] = p * B + r;
    __syncthreads();
    if (threadIdx.x == 0) base = b + n;
    __syncthreads();
  }
  if (threadIdx.x == 0) *n_out = base;
}

// One block per worker: n_sf of its directory entry = number of its u rows flagged nonzero (in a compacted stream
// the kept pairs are exactly the leading rows); block 0 sets the header's "compacted" flag.
__global__ void __launch_bounds__(256) count_pairs_kernel(const uint8_t* __restrict__ flags, int B, char* buf) {
  __shared__ int total;
  if (threadIdx.x == 0) total = 0;
  __syncthreads();
  const int p = blockIdx.x;
  int n = 0;
  for (int r = threadIdx.x; r < B; r += 256) n += flags[(size_t)p * B + r] != 0 ? 1 : 0;
  for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xffffffffu, n, o);
  if ((threadIdx.x & 31) == 0) atomicAdd(&total, n);   // integer: the order does not matter
  __syncthreads();
  if (threadIdx.x == 0) {
    reinterpret_cast<uint32_t*>(buf + 128 + (size_t)p * 32)[1] = (uint32_t)total;
    if (p == 0) reinterpret_cast<uint32_t*>(buf)[2] |= 2u;
  }
}

struct Scratch {
  uint8_t* flags; int* dest; int* counts;
};
// flags [K] bytes, new slots [K] ints, per-worker counts [P] ints; offsets fixed by the full K = P * B
Scratch scratch(void* workspace, int K) {
  Scratch w;
  w.flags = reinterpret_cast<uint8_t*>(workspace);
  w.dest = reinterpret_cast<int*>(reinterpret_cast<char*>(workspace) + pad_to(K, 256));
  w.counts = reinterpret_cast<int*>(reinterpret_cast<char*>(w.dest) + pad_to((long long)K * 4, 256));
  return w;
}

}  // namespace

long long compact_workspace_bytes(int K, int P) {
  return pad_to((long long)K, 256) + pad_to((long long)K * 4, 256) + pad_to((long long)P * 4, 256);
}

// Directory pair counts of a buffer whose streams were compacted elsewhere (each process of a sharded step compacts
// the streams of its own workers before the exchange; the directory is local and is rebuilt from what arrived).
int launch_count_pairs(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, void* workspace) {
  const int K = d.P * d.B;
  const Scratch w = scratch(workspace, K);
  char* buf = reinterpret_cast<char*>(sf_buf);
  RowMap u;
  u.base = buf + l.streams_off; u.worker_stride = l.stream_stride; u.ld = l.ldu; u.B = d.B; u.es = l.es;
  row_nonzero_kernel<<<(K + 7) / 8, 256, 0, s>>>(u, K, d.J, w.flags);
  count_pairs_kernel<<<d.P, 256, 0, s>>>(w.flags, d.B, buf);
  return cudaGetLastError() == cudaSuccess ? 2 : SFB_ERR_CUDA;
}

// first_worker / n_workers: compact only the streams of those workers (n_workers = 0: all P).  Worker indices
// inside the kernels are relative to first_worker: streams, directory entries, flags, slots and counts alike
// (counts[p] of the workspace belongs to worker first_worker + p).
int launch_compact(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, void* workspace, int first_worker,
                   int n_workers) {
  if (n_workers <= 0) { first_worker = 0; n_workers = d.P; }
  const int K = n_workers * d.B;
  const Scratch w = scratch(workspace, d.P * d.B);
  char* buf = reinterpret_cast<char*>(sf_buf);
  char* streams = buf + l.streams_off + (long long)first_worker * l.stream_stride;
  RowMap u;
  u.base = streams; u.worker_stride = l.stream_stride; u.ld = l.ldu; u.B = d.B; u.es = l.es;
  row_nonzero_kernel<<<(K + 7) / 8, 256, 0, s>>>(u, K, d.J, w.flags);
  compact_scan_kernel<<<n_workers, 256, 0, s>>>(w.flags, d.B, w.dest, w.counts, buf, first_worker);
  const int u_units = l.ldu * l.es / 16, v_units = l.ldv * l.es / 16;
  const int u_slices = (u_units + SLICE_UNITS - 1) / SLICE_UNITS, v_slices = (v_units + SLICE_UNITS - 1) / SLICE_UNITS;
  compact_move_kernel<<<dim3(n_workers, u_slices + v_slices), 256, 0, s>>>(streams, l.stream_stride, l.u_bytes, d.B, u_units,
                                                                           v_units, u_slices, w.dest, w.counts);
  return cudaGetLastError() == cudaSuccess ? 3 : SFB_ERR_CUDA;
}

int launch_kept_rows(cudaStream_t s, const void* sf_buf, int B, int workers, int* idx, int* n_out) {
  kept_rows_kernel<<<1, 256, 0, s>>>(reinterpret_cast<const char*>(sf_buf), B, workers, idx, n_out);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

}  // namespace sfb
