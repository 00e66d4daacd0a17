// Shared declarations of the SF hot-path kernels (internal; the public boundary is include/sfb.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sfb.h"

namespace sfb {

// Where the K factor rows of one operand live: row i of worker p = i / B sits at
// base + p * worker_stride + (i % B) * ld * elem_size.  Covers both caller-side [K][ld] arrays
// (worker_stride = B * ld * elem_size) and the U / V blocks of the SF buffer's worker streams.
struct RowMap {
  char* base;
  long long worker_stride;  // bytes
  int ld;                   // values per row (padded)
  int B;                    // rows per worker
  int es;                   // bytes per value (4 = fp32, 2 = bf16)
  __host__ __device__ __forceinline__ char* row(int i) const {
    return base + (long long)(i / B) * worker_stride + (long long)(i % B) * ld * es;
  }
};

// Byte layout of the SF buffer for one descriptor (see the wire format in include/sfb.h).
struct Layout {
  int es, ldu, ldv, cap_p;
  long long u_bytes, v_bytes, rp_bytes, idx_bytes, val_bytes;
  long long stream_stride, streams_off, total_bytes;
};

static inline long long pad_to(long long n, long long a) { return (n + a - 1) / a * a; }

// Optional extra outputs of a kernel that writes fp32 factor rows on the compensated tf32 path: the rows'
// bf16 correction operands (split.cu), so that no separate pass has to read the rows again.
//   mn: for the apply (MN-major), [block of 32 pairs][64 lines][ldc]; pair (worker w, row r) sits in block
//       w * k_bpw + r / 32, line r % 32 (k_wp == 1: whole blocks per worker), or in block w / k_wp, line
//       (w % k_wp) * k_bb + r (k_bb rows of each of k_wp workers per block); a_side: remainder lines first.
//   km: for the forward (K-major A side), [pair][atom][32 remainders | 32 values].
struct CorrOut {
  char* mn;
  char* km;
  int ldc, k_bb, k_wp, k_bpw, a_side, atoms;
  __host__ __device__ CorrOut() : mn(nullptr), km(nullptr), ldc(0), k_bb(32), k_wp(1), k_bpw(1), a_side(0), atoms(0) {}
};
#ifdef __CUDACC__
// values t of pair i (B pairs per worker) at columns j .. j + 3, j a multiple of 4
__device__ __forceinline__ void corr_store4(const CorrOut& c, int i, int B, int j, float4 t) {
  const float rx = t.x - __uint_as_float(__float_as_uint(t.x) & 0xFFFFE000u);
  const float ry = t.y - __uint_as_float(__float_as_uint(t.y) & 0xFFFFE000u);
  const float rz = t.z - __uint_as_float(__float_as_uint(t.z) & 0xFFFFE000u);
  const float rw = t.w - __uint_as_float(__float_as_uint(t.w) & 0xFFFFE000u);
  const __nv_bfloat162 v0 = __floats2bfloat162_rn(t.x, t.y), v1 = __floats2bfloat162_rn(t.z, t.w);
  const __nv_bfloat162 r0 = __floats2bfloat162_rn(rx, ry), r1 = __floats2bfloat162_rn(rz, rw);
  const uint2 val = make_uint2(*reinterpret_cast<const uint32_t*>(&v0), *reinterpret_cast<const uint32_t*>(&v1));
  const uint2 rem = make_uint2(*reinterpret_cast<const uint32_t*>(&r0), *reinterpret_cast<const uint32_t*>(&r1));
  if (c.mn != nullptr && j < c.ldc) {
    const int w = i / B, r = i - w * B;
    long long blk;
    int line;
    if (c.k_wp == 1) { blk = (long long)w * c.k_bpw + (r >> 5); line = r & 31; }
    else { blk = w / c.k_wp; line = (w % c.k_wp) * c.k_bb + r; }
    char* base = c.mn + ((blk * 64) * c.ldc + j) * 2;
    *reinterpret_cast<uint2*>(base + (long long)(c.a_side ? line : 32 + line) * c.ldc * 2) = rem;
    *reinterpret_cast<uint2*>(base + (long long)(c.a_side ? 32 + line : line) * c.ldc * 2) = val;
  }
  if (c.km != nullptr && (j >> 5) < c.atoms) {
    char* atom = c.km + (((long long)i * c.atoms + (j >> 5)) * 64 + (j & 31)) * 2;
    *reinterpret_cast<uint2*>(atom) = rem;
    *reinterpret_cast<uint2*>(atom + 64) = val;
  }
}
#endif

static inline Layout make_layout(const sfb_desc& d) {
  Layout l;
  l.es = (d.path == SFB_PATH_BF16) ? 2 : 4;
  const int unit = 16 / l.es;
  l.ldu = (int)pad_to(d.J, unit);
  l.ldv = (int)pad_to(d.D, unit);
  l.cap_p = d.v_sparse ? (int)(d.nnz_capacity / (uint64_t)d.P) : 0;
  l.u_bytes = pad_to((long long)d.B * l.ldu * l.es, 128);
  if (d.v_sparse) {
    l.rp_bytes = pad_to((long long)(d.B + 1) * 4, 128);
    l.idx_bytes = pad_to((long long)l.cap_p * 4, 128);
    l.val_bytes = pad_to((long long)l.cap_p * l.es, 128);
    l.v_bytes = l.rp_bytes + l.idx_bytes + l.val_bytes;
  } else {
    l.rp_bytes = l.idx_bytes = l.val_bytes = 0;
    l.v_bytes = pad_to((long long)d.B * l.ldv * l.es, 128);
  }
  l.stream_stride = l.u_bytes + l.v_bytes;
  l.streams_off = 128 + pad_to((long long)d.P * 32, 128);
  l.total_bytes = l.streams_off + (long long)d.P * l.stream_stride;
  return l;
}

// cudaFuncSetAttribute acts on the current device only: first() is true once per device (ordinals 0..63)
// for the static object it is called on.  A repeated call from a racing thread would set the same value.
struct PerDeviceOnce {
  unsigned long long done = 0;
  bool first() {
    int dev = 0;
    cudaGetDevice(&dev);
    const unsigned long long bit = 1ull << (dev & 63);
    if (done & bit) return false;
    done |= bit;
    return true;
  }
};

// ---- kernel launchers (each returns the number of kernels it launched, or a negative SFB_ERR_*) ----

// Z[i][j] = sum_d A[i][d] * W[j][d] on fp32 CUDA cores, written as fp32 rows through `z`.
// A = X, or X - Xb (element-wise fp32 subtraction) when Xb != nullptr.  When `v` has a base, the
// operand rows (X, or the difference) are also written there (the factor v), pad columns zero.
// With a `part` row map (fp32 rows, split_stride bytes between partial buffers) and nsplit_out, a problem
// with few tiles has its reduction cut into *nsplit_out ranges whose partial products go to `part` instead
// of `z` (the finishing pass sums them in range order); forward_f32_splits tells how many in advance.
// v rows = Xa rows - Xb rows, one fp32 subtraction per element, pad columns zero (the DML factor v).
int launch_diff_rows(cudaStream_t s, const float* Xa, const float* Xb, RowMap v, int K, int D, CorrOut corr = CorrOut());
int forward_f32_splits(int K, int J, int D);
// The same contraction through transposed copies of both operands (two transposing passes, then the pipelined
// large-tile kernel).  src: operand rows a_i behind a row map; copy (optional): those rows also written there;
// ws: forward_f32_nn_workspace_floats(K, J, D) floats.  Needs at least one full 128 x 128 tile of work to pay.
long long forward_f32_nn_workspace_floats(int K, int J, int D);
int launch_forward_f32_nn(cudaStream_t s, const float* W, RowMap src, RowMap copy, int K, int J, int D, float* ws,
                          RowMap z, RowMap part, long long split_stride, int max_splits, int* nsplit_out);
int launch_forward_f32(cudaStream_t s, const float* W, const float* X, const float* Xb, int K, int J, int D,
                       RowMap z, RowMap v, RowMap part = RowMap(), long long split_stride = 0, int max_splits = 1,
                       int* nsplit_out = nullptr);

// W[j][d] -= eta * sum_{i<K} U[i][j] * V[i][d] on fp32 CUDA cores (fixed summation order).
int launch_apply_f32(cudaStream_t s, float* W, RowMap u, RowMap v, int K, int J, int D, float eta,
                     const int* dev_status, const int* row_idx = nullptr, const int* n_rows = nullptr);
// row_idx / n_rows (optional, device): apply only the factor rows row_idx[0 .. *n_rows), in that order, instead of
// rows 0 .. K-1 (rows that are known to be all zeros can be left out: the result is bit-identical).

// MLR epilogue: u = softmax(z) - onehot(label).  z rows are fp32; u rows fp32 or bf16 (u.es).
// z may be `nsplit` partial products (split s at z + s * split_stride_bytes), summed in split order.
// dual (optional, SDCA): fp32 dual variables of the K samples, [K][J rounded up to 4], updated in place; the factor
// written to u is then the dual step sdca_step * (dual + softmax - onehot).
int launch_finish_mlr(cudaStream_t s, RowMap z, RowMap u, const int32_t* labels, int K, int J, int* dev_status,
                      int nsplit = 1, long long split_stride_bytes = 0, float* dual = nullptr, float sdca_step = 0.f,
                      CorrOut corr = CorrOut());

// DML epilogue: u = +z (similar) or -z * [|z|^2 < margin] (dissimilar).
// active (optional, [K] bytes): 1 where the pair contributes (similar, or dissimilar inside the margin), 0 where u_i = 0.
int launch_finish_dml(cudaStream_t s, RowMap z, RowMap u, const uint8_t* similar, float margin, int K, int J,
                      int nsplit = 1, long long split_stride_bytes = 0, uint8_t* active = nullptr, CorrOut corr = CorrOut());
// idx[0 .. *n_out) = ascending list of the samples i < K with active[i] != 0 (device arrays; one ordered block).
int launch_compact_active(cudaStream_t s, const uint8_t* active, int K, int* idx, int* n_out);

// Copies K rows of `cols` values from src to dst rows (same value type), zero-filling dst pad columns.
int launch_copy_rows(cudaStream_t s, RowMap src, RowMap dst, int K, int cols, CorrOut corr = CorrOut());

// Writes header and directory of the SF buffer.  `rowptr` (global CSR row pointers) only for sparse v.
int launch_write_header(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, uint32_t clock,
                        const uint32_t* rowptr);

// Copies the CSR codes of every worker into its stream (local row pointers, zero-filled tail).
int launch_pack_csr(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, const uint32_t* rowptr,
                    const uint32_t* idx, const float* val, int* dev_status);

// Inactive-pair compaction of a committed dense-v buffer, in place: per worker the pairs with a nonzero u move to
// the front (same order), the slots behind them are cleared, the directory gets the pair counts and the header
// its "compacted" flag.  workspace: compact_workspace_bytes(K, P) bytes.  launch_kept_rows lists the slots
// p * B + r, r < count of worker p, of the first `workers` workers (idx [K], n_out one int; device arrays).
long long compact_workspace_bytes(int K, int P);
int launch_compact(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, void* workspace, int first_worker = 0,
                   int n_workers = 0);   // n_workers > 0: only those workers' streams (a process's shard)
// Rebuilds the directory's pair counts (and the header flag) from streams that arrived already compacted.
int launch_count_pairs(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, void* workspace);
int launch_kept_rows(cudaStream_t s, const void* sf_buf, int B, int workers, int* idx, int* n_out);

// Sets SFB_DEV_BAD_HEADER in *dev_status unless the buffer's header matches the descriptor.
int launch_check_header(cudaStream_t s, const void* sf_buf, const sfb_desc& d, const Layout& l, int* dev_status);

// SC forward: u_i = sum_{(d,a) in code i} a * W[:, d] - x_i, codes read from CSR arrays whose row
// pointers are either global ([K+1]) or per worker stream inside the SF buffer.
struct CsrView {
  const char* base;          // SF buffer base, or nullptr for caller-side global arrays
  const uint32_t* rowptr;    // global arrays (base == nullptr)
  const uint32_t* idx;
  const float* val;
  long long streams_off, stream_stride, v_off, rp_bytes, idx_bytes;  // stream-relative offsets (base != nullptr)
  int B;
  int cap_p;                 // global arrays only: > 0 cuts every worker's rows off after its first cap_p nonzeros
                             // (what pack_csr keeps in the stream); 0 = rows as given
};
// Wt is a caller-provided workspace of sc_forward_workspace_bytes(J, D) bytes (atom-major copy of W).
long long sc_forward_workspace_bytes(int J, int D);
int launch_sc_forward_ws(cudaStream_t s, const float* W, float* Wt, CsrView codes, const float* Xdata, RowMap u, int K,
                         int J, int D, int* dev_status);

// SC apply: W[:, d] -= eta * sum_{i: a_id != 0} a_id * u_i (sparse-v scatter, no float atomics).
int launch_sc_apply(cudaStream_t s, float* W, CsrView codes, RowMap u, int K, int J, int D, float eta,
                    const int* dev_status_ro, int* dev_status);

// The same update through an atom-major (CSC) re-sort of the codes and shared-memory u columns (faster;
// needs sc_csc_supported(K) and a workspace of sc_csc_workspace_bytes(K, D, nnz_capacity) bytes).
long long sc_csc_workspace_bytes(int K, int D, long long nnz_capacity);
bool sc_csc_supported(int K);
int launch_sc_apply_csc(cudaStream_t s, float* W, CsrView codes, RowMap u, int K, int J, int D, float eta,
                        long long nnz_capacity, void* workspace, const int* dev_status_ro);
// The two halves of launch_sc_apply_csc: the re-sort reads only the codes (it can run beside the forward
// pass), the update needs u and the workspace the re-sort filled.
// dev_status (optional): SFB_DEV_BAD_INDEX is set for entries the re-sort leaves out (atom out of range, row not
// strictly ascending: the same entries the forward pass skips).
int launch_sc_csc_build(cudaStream_t s, CsrView codes, int K, int D, long long nnz_capacity, void* workspace,
                        int* dev_status = nullptr);
int launch_sc_csc_apply(cudaStream_t s, float* W, RowMap u, int K, int J, int D, float eta, long long nnz_capacity,
                        void* workspace, const int* dev_status_ro);

// Dense fp32 rows a_i of the CSR codes (zeros elsewhere), for the tensor-core sparse-coding path.
// round_tf32: values rounded to the nearest tf32 (the plain tf32 path, whose tensor cores would truncate them).
int launch_densify_codes(cudaStream_t s, CsrView codes, RowMap a, int K, int D, int* dev_status, bool round_tf32 = true);
// The same (exact values) with the rows' correction operands written beside them; a row of ld floats must fit in
// shared memory (densify_corr_fits).
bool densify_corr_fits(int ld);
int launch_densify_codes_corr(cudaStream_t s, CsrView codes, RowMap a, int K, int D, int* dev_status, CorrOut corr);

// SC epilogue on dense products: u = z - x in place (u rows hold z), pad columns zero.
// z: products (possibly `nsplit` partials); u = sum of partials - x.
int launch_finish_sc(cudaStream_t s, RowMap z, RowMap u, const float* Xdata, int K, int J, int nsplit = 1,
                     long long split_stride_bytes = 0, CorrOut corr = CorrOut());

// Column-norm projection: every column of W with 2-norm above 1 is divided by its norm (in place).
int launch_prox_unit_columns(cudaStream_t s, float* W, int J, int D);
// Minibatch objective: per-sample values from the fp32 rows (z_i for MLR / DML, u_i for SC) into loss_i[K],
// then their fp64 sum into *total (device).  Two launches.
int launch_sample_loss(cudaStream_t s, int model, RowMap rows, const int32_t* labels, const uint8_t* similar, float margin,
                       int K, int J, float* loss_i, double* total, int* dev_status);

// W (fp32) -> bf16 shadow, round to nearest even.
int launch_cast_bf16(cudaStream_t s, const float* W, __nv_bfloat16* Wb, long long n);
// Correction operands of the error-compensated tf32 kernels (split.cu): bf16 [remainder | value] (A side) or
// [value | remainder] (B side) of fp32 rows.  K-major: dst[row][atom][64] over `rows` rows of `cols` values.
// MN-major: dst[block][64][ldc], block = 32 pairs taken as the apply's reduction blocks are (32 rows of one
// worker, or k_bb rows of each of k_wp workers), ldc a multiple of 64.
int launch_split_k(cudaStream_t s, RowMap src, int rows, int cols, void* dst, bool a_side);
int launch_split_mn(cudaStream_t s, RowMap src, int cols, int workers, int k_bb, int k_wp, int k_bpw, int blocks,
                    void* dst, int ldc, bool a_side);

}  // namespace sfb
