// fp32 CUDA-core contractions of the SF hot path.
//
//   forward:  Z[i][j] = sum_d A[i][d] * W[j][d]      (z_i = W a_i for every sample; Section 2, (P))
//   apply  :  W[j][d] -= eta * sum_i U[i][j] * V[i][d]  (W <- W - eta * sum_i u_i v_i^T; Section 3)
//
// Both are register-blocked shared-memory SGEMMs: 256 threads, a (64*MI) x (64*NI) output tile, a
// reduction step of 16, operands staged k-major in shared memory so that every inner-loop read is
// a conflict-free 16-byte load, global loads prefetched into registers one step ahead.  The
// summation order is fixed (ascending reduction index inside one thread), so results are
// bit-reproducible run to run.
#include "common.cuh"

namespace sfb {
namespace {

constexpr int BK = 16;

__device__ __forceinline__ float4 ld4_guard(const float* row, int c, int cols, bool vec_ok) {
  // row: start of a row; c: first column (multiple of 4); cols: valid columns
  if (vec_ok && c + 3 < cols) return *reinterpret_cast<const float4*>(row + c);
  float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
  if (c < cols) r.x = row[c];
  if (c + 1 < cols) r.y = row[c + 1];
  if (c + 2 < cols) r.z = row[c + 2];
  if (c + 3 < cols) r.w = row[c + 3];
  return r;
}

// PACKED: the multiply-adds as packed fp32 pairs (two independent round-to-nearest FMAs per instruction: half
// the issue slots of scalar FFMA for the same arithmetic, bit-identical results).  It pays in the apply kernels;
// the forward kernel, which also holds its operand prefetch in registers, measured slower with it.
template <int MI, int NI, bool PACKED>
__device__ __forceinline__ void mma_tile(const float (*As)[64 * MI + 4], const float (*Bs)[64 * NI + 4], int ty,
                                         int tx, float2 (&acc)[4 * MI][2 * NI]) {
#pragma unroll
  for (int k = 0; k < BK; ++k) {
    float a[4 * MI], b[4 * NI];
#pragma unroll
    for (int mi = 0; mi < MI; ++mi) {
      float4 t = *reinterpret_cast<const float4*>(&As[k][mi * 64 + ty * 4]);
      a[mi * 4 + 0] = t.x; a[mi * 4 + 1] = t.y; a[mi * 4 + 2] = t.z; a[mi * 4 + 3] = t.w;
    }
#pragma unroll
    for (int ni = 0; ni < NI; ++ni) {
      float4 t = *reinterpret_cast<const float4*>(&Bs[k][ni * 64 + tx * 4]);
      b[ni * 4 + 0] = t.x; b[ni * 4 + 1] = t.y; b[ni * 4 + 2] = t.z; b[ni * 4 + 3] = t.w;
    }
#pragma unroll
    for (int m = 0; m < 4 * MI; ++m) {
      const float2 aa = make_float2(a[m], a[m]);
#pragma unroll
      for (int n = 0; n < 2 * NI; ++n) {
        if (PACKED) {
          acc[m][n] = __ffma2_rn(aa, make_float2(b[2 * n], b[2 * n + 1]), acc[m][n]);
        } else {
          acc[m][n].x = fmaf(a[m], b[2 * n], acc[m][n].x);
          acc[m][n].y = fmaf(a[m], b[2 * n + 1], acc[m][n].y);
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------ forward
// Tile rows = samples i (BM = 64*MI), tile columns = classes j (BN = 64*NI), reduction over d.
// Both operands are contiguous along d, so tiles are transposed while being stored to shared memory.
template <int MI, int NI>
__global__ void __launch_bounds__(256, 2) forward_f32_kernel(const float* __restrict__ W, const float* __restrict__ X,
                                                          const float* __restrict__ Xb, int K, int J, int D,
                                                          RowMap z, RowMap v, int d_per_split, long long split_stride) {
  constexpr int BM = 64 * MI, BN = 64 * NI;
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  const bool vec_ok = (D & 3) == 0;
  const bool write_v = (v.base != nullptr) && (blockIdx.x == 0);
  const int lr = tid >> 2, lc = (tid & 3) * 4;   // loader: row within 64, first of 4 reduction columns

  float2 acc[4 * MI][2 * NI];
#pragma unroll
  for (int m = 0; m < 4 * MI; ++m)
#pragma unroll
    for (int n = 0; n < 2 * NI; ++n) acc[m][n] = make_float2(0.f, 0.f);

  float4 pa[MI], pb[NI];
  auto fetch = [&](int d0) {
#pragma unroll
    for (int q = 0; q < MI; ++q) {
      const int i = i0 + lr + 64 * q;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i < K) {
        a = ld4_guard(X + (size_t)i * D, d0 + lc, D, vec_ok);
        if (Xb != nullptr) {
          const float4 b = ld4_guard(Xb + (size_t)i * D, d0 + lc, D, vec_ok);
          a.x = __fsub_rn(a.x, b.x); a.y = __fsub_rn(a.y, b.y); a.z = __fsub_rn(a.z, b.z); a.w = __fsub_rn(a.w, b.w);
        }
        if (write_v && d0 + lc < v.ld) *reinterpret_cast<float4*>(v.row(i) + (size_t)(d0 + lc) * 4) = a;
      }
      pa[q] = a;
    }
#pragma unroll
    for (int q = 0; q < NI; ++q) {
      const int j = j0 + lr + 64 * q;
      pb[q] = (j < J) ? ld4_guard(W + (size_t)j * D, d0 + lc, D, vec_ok) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int q = 0; q < MI; ++q) {
      As[lc + 0][lr + 64 * q] = pa[q].x; As[lc + 1][lr + 64 * q] = pa[q].y;
      As[lc + 2][lr + 64 * q] = pa[q].z; As[lc + 3][lr + 64 * q] = pa[q].w;
    }
#pragma unroll
    for (int q = 0; q < NI; ++q) {
      Bs[lc + 0][lr + 64 * q] = pb[q].x; Bs[lc + 1][lr + 64 * q] = pb[q].y;
      Bs[lc + 2][lr + 64 * q] = pb[q].z; Bs[lc + 3][lr + 64 * q] = pb[q].w;
    }
  };

  // blockIdx.z takes the reduction range [d_lo, d_hi) and writes its partial products split_stride bytes
  // after the previous range's (one range: the whole reduction, written to z itself)
  const int d_lo = blockIdx.z * d_per_split;
  const int d_hi = min(D, d_lo + d_per_split);
  fetch(d_lo);
  for (int d0 = d_lo; d0 < d_hi; d0 += BK) {
    stash();
    __syncthreads();
    if (d0 + BK < d_hi) fetch(d0 + BK);
    mma_tile<MI, NI, false>(As, Bs, ty, tx, acc);
    __syncthreads();
  }
  // The factor v has pad columns [D, ldv): the last loader step wrote zeros there only when
  // D..ldv falls inside a fetched float4, which holds because ldv = D rounded up to 4.

#pragma unroll
  for (int mi = 0; mi < MI; ++mi)
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int i = i0 + mi * 64 + ty * 4 + a;
      if (i >= K) continue;
      float* zr = reinterpret_cast<float*>(z.row(i) + blockIdx.z * split_stride);
#pragma unroll
      for (int ni = 0; ni < NI; ++ni) {
        const int j = j0 + ni * 64 + tx * 4;
        if (j < z.ld)   // ld is a multiple of 4, so the whole float4 is inside the row; columns >= J hold 0
          *reinterpret_cast<float4*>(zr + j) = make_float4(acc[mi * 4 + a][ni * 2].x, acc[mi * 4 + a][ni * 2].y,
                                                           acc[mi * 4 + a][ni * 2 + 1].x, acc[mi * 4 + a][ni * 2 + 1].y);
      }
    }
}

// ------------------------------------------------------------------------------------------ apply
// Tile rows = rows j of W (BM), tile columns = columns d of W (BN), reduction over the K factors.
// U rows are contiguous along j and V rows along d: tiles go to shared memory as they are.
template <int MI, int NI>
__global__ void __launch_bounds__(256, 2) apply_f32_kernel(float* __restrict__ W, RowMap u, RowMap v, int K, int J,
                                                        int D, float eta, const int* __restrict__ dev_status) {
  constexpr int BM = 64 * MI, BN = 64 * NI;
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  if (dev_status != nullptr && (*dev_status & SFB_DEV_BAD_HEADER)) return;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int j0 = blockIdx.y * BM, d0 = blockIdx.x * BN;
  const int lr = tid >> 4, lc = (tid & 15) * 4;   // loader: factor row within 16, first of 4 columns

  float2 acc[4 * MI][2 * NI];
#pragma unroll
  for (int m = 0; m < 4 * MI; ++m)
#pragma unroll
    for (int n = 0; n < 2 * NI; ++n) acc[m][n] = make_float2(0.f, 0.f);

  float4 pa[MI], pb[NI];
  auto fetch = [&](int k0) {
    const int i = k0 + lr;
#pragma unroll
    for (int q = 0; q < MI; ++q) {
      const int j = j0 + lc + 64 * q;
      pa[q] = (i < K) ? ld4_guard(reinterpret_cast<const float*>(u.row(i)), j, J, true)
                      : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int q = 0; q < NI; ++q) {
      const int d = d0 + lc + 64 * q;
      pb[q] = (i < K) ? ld4_guard(reinterpret_cast<const float*>(v.row(i)), d, D, true)
                      : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int q = 0; q < MI; ++q) *reinterpret_cast<float4*>(&As[lr][lc + 64 * q]) = pa[q];
#pragma unroll
    for (int q = 0; q < NI; ++q) *reinterpret_cast<float4*>(&Bs[lr][lc + 64 * q]) = pb[q];
  };

  fetch(0);
  for (int k0 = 0; k0 < K; k0 += BK) {
    stash();
    __syncthreads();
    if (k0 + BK < K) fetch(k0 + BK);
    mma_tile<MI, NI, true>(As, Bs, ty, tx, acc);
    __syncthreads();
  }

  const bool vec_ok = (D & 3) == 0;
#pragma unroll
  for (int mi = 0; mi < MI; ++mi)
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int j = j0 + mi * 64 + ty * 4 + a;
      if (j >= J) continue;
      float* wr = W + (size_t)j * D;
#pragma unroll
      for (int ni = 0; ni < NI; ++ni) {
        const int d = d0 + ni * 64 + tx * 4;
        const float c[4] = {acc[mi * 4 + a][ni * 2].x, acc[mi * 4 + a][ni * 2].y, acc[mi * 4 + a][ni * 2 + 1].x,
                            acc[mi * 4 + a][ni * 2 + 1].y};
        if (vec_ok && d + 3 < D) {
          float4 w = *reinterpret_cast<float4*>(wr + d);
          w.x = fmaf(-eta, c[0], w.x); w.y = fmaf(-eta, c[1], w.y);
          w.z = fmaf(-eta, c[2], w.z); w.w = fmaf(-eta, c[3], w.w);
          *reinterpret_cast<float4*>(wr + d) = w;
        } else {
#pragma unroll
          for (int b = 0; b < 4; ++b)
            if (d + b < D) wr[d + b] = fmaf(-eta, c[b], wr[d + b]);
        }
      }
    }
}

// ---- large tiles with operands whose rows run along the OUTPUT indices: C[m][n] (+)= sum_k A[k][m] * B[k][n].
// The rows go to shared memory as they are, fetched with 16-byte asynchronous copies (zero-filled beyond the
// reduction range, M and N) through a ring of PIPE stages: one barrier per reduction step, no staging registers.
//   OUT 0 (apply):   A = factor rows u_i (k = sample, m = row j of W), B = v_i; W[m][n] -= eta * C[m][n].
//   OUT 1 (forward): A = X^T (k = feature d, m = sample i), B = W^T (n = class j), both made by a transposing
//                    pass; the products of reduction range blockIdx.z are stored to z rows (+ range stride).
constexpr int PIPE = 4;
constexpr int PIPE_STAGE_FLOATS = 2 * BK * (128 + 4);

__device__ __forceinline__ void cp_async16_zfill(float* dst_smem, const void* src, int src_bytes) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst_smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int OUT>
__global__ void __launch_bounds__(256, 2) sgemm_pipe_kernel(float* __restrict__ W, RowMap u, RowMap v, int K, int J,
                                                         int D, float eta, const int* __restrict__ dev_status,
                                                         RowMap z, int k_per_range, long long range_stride,
                                                         const int* __restrict__ row_idx, const int* __restrict__ n_rows) {
  constexpr int BM = 128, BN = 128;
  extern __shared__ __align__(16) float ring[];
  if (OUT == 0 && dev_status != nullptr && (*dev_status & SFB_DEV_BAD_HEADER)) return;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int j0 = blockIdx.y * BM, d0 = blockIdx.x * BN;
  const int k_lo = (OUT == 1) ? blockIdx.z * k_per_range : 0;
  // OUT 0 with a row list: the reduction runs over the listed factor rows only (the others are all zeros)
  const int k_hi = (OUT == 1) ? min(K, k_lo + k_per_range) : (n_rows != nullptr ? min(K, *n_rows) : K);
  const int lr = tid >> 5, lc = (tid & 31) * 4;   // loader: factor rows lr and lr + 8 of the step, 4 columns at lc
  // bytes of this thread's 16-byte piece that exist (the rest is zero-filled); a piece with nothing to read
  // still needs a valid aligned address: column 0 of a valid row
  const int ju = j0 + lc, dv = d0 + lc;
  const int u_bytes = max(0, min(16, (J - ju) * 4)), v_bytes = max(0, min(16, (D - dv) * 4));
  const size_t u_off = u_bytes > 0 ? (size_t)ju * 4 : 0, v_off = v_bytes > 0 ? (size_t)dv * 4 : 0;

  auto issue = [&](int stage, int k0) {
    float* As = ring + stage * PIPE_STAGE_FLOATS;
    float* Bs = As + BK * (BM + 4);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int r = lr + 8 * h, i = k0 + r;
      const bool ok = i < k_hi;
      const int ii = ok ? ((OUT == 0 && row_idx != nullptr) ? row_idx[i] : i) : 0;
      cp_async16_zfill(As + r * (BM + 4) + lc, u.row(ii) + u_off, ok ? u_bytes : 0);
      cp_async16_zfill(Bs + r * (BN + 4) + lc, v.row(ii) + v_off, ok ? v_bytes : 0);
    }
  };

  float2 acc[8][4];
#pragma unroll
  for (int m = 0; m < 8; ++m)
#pragma unroll
    for (int n = 0; n < 4; ++n) acc[m][n] = make_float2(0.f, 0.f);

  const int nk = (k_hi - k_lo + BK - 1) / BK;
#pragma unroll
  for (int st = 0; st < PIPE - 1; ++st) {
    if (st < nk) issue(st, k_lo + st * BK);
    cp_async_commit();
  }
  for (int kt = 0; kt < nk; ++kt) {
    cp_async_wait<PIPE - 2>();       // this thread's pieces of step kt have landed
    __syncthreads();                 // ... everybody's have, and everybody is done with step kt - 1
    const int nxt = kt + PIPE - 1;
    if (nxt < nk) issue(nxt % PIPE, k_lo + nxt * BK);
    cp_async_commit();
    const float* As = ring + (kt % PIPE) * PIPE_STAGE_FLOATS;
    mma_tile<2, 2, true>(reinterpret_cast<const float(*)[BM + 4]>(As), reinterpret_cast<const float(*)[BN + 4]>(As + BK * (BM + 4)),
                   ty, tx, acc);
  }
  cp_async_wait<0>();

  if (OUT == 1) {   // rows of z: m = sample, n = class; z.ld is a multiple of 4 and columns J .. z.ld - 1 get zeros
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int i = j0 + mi * 64 + ty * 4 + a;
        if (i >= J) continue;
        float* zr = reinterpret_cast<float*>(z.row(i) + blockIdx.z * range_stride);
#pragma unroll
        for (int ni = 0; ni < 2; ++ni) {
          const int n = d0 + ni * 64 + tx * 4;
          if (n < z.ld)
            *reinterpret_cast<float4*>(zr + n) = make_float4(acc[mi * 4 + a][ni * 2].x, acc[mi * 4 + a][ni * 2].y,
                                                             acc[mi * 4 + a][ni * 2 + 1].x, acc[mi * 4 + a][ni * 2 + 1].y);
        }
      }
    return;
  }

  const bool vec_ok = (D & 3) == 0;
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int j = j0 + mi * 64 + ty * 4 + a;
      if (j >= J) continue;
      float* wr = W + (size_t)j * D;
#pragma unroll
      for (int ni = 0; ni < 2; ++ni) {
        const int d = d0 + ni * 64 + tx * 4;
        const float c[4] = {acc[mi * 4 + a][ni * 2].x, acc[mi * 4 + a][ni * 2].y, acc[mi * 4 + a][ni * 2 + 1].x,
                            acc[mi * 4 + a][ni * 2 + 1].y};
        if (vec_ok && d + 3 < D) {
          float4 w = *reinterpret_cast<float4*>(wr + d);
          w.x = fmaf(-eta, c[0], w.x); w.y = fmaf(-eta, c[1], w.y);
          w.z = fmaf(-eta, c[2], w.z); w.w = fmaf(-eta, c[3], w.w);
          *reinterpret_cast<float4*>(wr + d) = w;
        } else {
#pragma unroll
          for (int b = 0; b < 4; ++b)
            if (d + b < D) wr[d + b] = fmaf(-eta, c[b], wr[d + b]);
        }
      }
    }
}

// dst[c][r] = src row r, column c (R rows of C values behind a row map; dst rows ldr floats long, columns R .. ldr - 1
// zero).  `copy` (optional): the same rows also copied there, pad columns zero (the factor v = x of the MLR model).
__global__ void __launch_bounds__(256) transpose_rows_kernel(RowMap src, float* __restrict__ dst, int R, int C, int ldr,
                                                             RowMap copy) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
#pragma unroll
  for (int q = 0; q < 32; q += 8) {
    const int r = r0 + ty + q, c = c0 + tx;
    float val = 0.f;
    if (r < R && c < C) val = reinterpret_cast<const float*>(src.row(r))[c];
    tile[ty + q][tx] = val;
    if (copy.base != nullptr && r < R && c < copy.ld) reinterpret_cast<float*>(copy.row(r))[c] = val;
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 32; q += 8) {
    const int c = c0 + ty + q, r = r0 + tx;
    if (c < C && r < ldr) dst[(size_t)c * ldr + r] = tile[tx][ty + q];
  }
}

// The same transposition for rows that are whole numbers of 16-byte units (C a multiple of 4, rows 16-byte aligned):
// 64 x 64 tiles, 16-byte global loads and stores on both sides, and both operands of the forward pass in one launch
// (blockIdx.z picks the job).
struct TransposeJob {
  RowMap src;
  float* dst;
  int R, C, ldr;
  RowMap copy;
};
__global__ void __launch_bounds__(256) transpose_rows_vec_kernel(TransposeJob j0, TransposeJob j1) {
  __shared__ float tile[64][65];
  const TransposeJob& j = blockIdx.z == 0 ? j0 : j1;
  const int c0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
  if (c0 >= j.C || r0 >= j.ldr) return;
  const int tq = threadIdx.x & 15, tr = threadIdx.x >> 4;   // 16 x 16
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int rr = tr + 16 * q, r = r0 + rr, c = c0 + tq * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < j.R && c < j.C) {
      v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(j.src.row(r)) + c);
      if (j.copy.base != nullptr) *reinterpret_cast<float4*>(reinterpret_cast<float*>(j.copy.row(r)) + c) = v;
    }
    tile[rr][tq * 4] = v.x; tile[rr][tq * 4 + 1] = v.y; tile[rr][tq * 4 + 2] = v.z; tile[rr][tq * 4 + 3] = v.w;
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int cc = tr + 16 * q, c = c0 + cc, r = r0 + tq * 4;
    if (c < j.C && r < j.ldr)
      *reinterpret_cast<float4*>(j.dst + (size_t)c * j.ldr + r) =
          make_float4(tile[tq * 4][cc], tile[tq * 4 + 1][cc], tile[tq * 4 + 2][cc], tile[tq * 4 + 3][cc]);
  }
}

}  // namespace

// Few 128 x 128 tiles and a long reduction (e.g. 1024 samples x 1000 classes over 20000 features): the
// reduction is cut into ranges so that the blocks fill whole waves of two blocks per SM.  Among 1 .. 12 ranges
// (each at least 512 reduction steps long) the smallest count whose last wave is at least 94 % full is taken,
// else the count with the fullest waves.
int forward_f32_splits(int K, int J, int D) {
  const long long tiles = (long long)((K + 127) / 128) * ((J + 127) / 128);
  const long long slots = 2 * 148;
  if (tiles >= 148) return 1;
  int best = 1;
  double best_fill = 0.0;
  for (int ks = 1; ks <= 12 && D / ks >= 512; ++ks) {
    const long long blocks = tiles * ks;
    const double fill = (double)blocks / (double)(((blocks + slots - 1) / slots) * slots);
    if (fill >= 0.94) return ks;
    if (fill > best_fill + 1e-9) { best_fill = fill; best = ks; }
  }
  return best;
}

int launch_forward_f32(cudaStream_t s, const float* W, const float* X, const float* Xb, int K, int J, int D,
                       RowMap z, RowMap v, RowMap part, long long split_stride, int max_splits, int* nsplit_out) {
  if (nsplit_out != nullptr) *nsplit_out = 1;
  const long long big_tiles = (long long)((K + 127) / 128) * ((J + 127) / 128);
  int ks = (part.base != nullptr && nsplit_out != nullptr) ? forward_f32_splits(K, J, D) : 1;
  if (ks > max_splits) ks = max_splits;       // the partial buffers the caller owns
  if (ks > 1) {
    const int per = ((D + ks - 1) / ks + BK - 1) / BK * BK;
    dim3 grid((J + 127) / 128, (K + 127) / 128, ks);
    forward_f32_kernel<2, 2><<<grid, 256, 0, s>>>(W, X, Xb, K, J, D, part, v, per, split_stride);
    *nsplit_out = ks;
  } else if (big_tiles >= 148) {
    dim3 grid((J + 127) / 128, (K + 127) / 128);
    forward_f32_kernel<2, 2><<<grid, 256, 0, s>>>(W, X, Xb, K, J, D, z, v, D, 0);
  } else {
    dim3 grid((J + 63) / 64, (K + 63) / 64);
    forward_f32_kernel<1, 1><<<grid, 256, 0, s>>>(W, X, Xb, K, J, D, z, v, D, 0);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_apply_f32(cudaStream_t s, float* W, RowMap u, RowMap v, int K, int J, int D, float eta,
                     const int* dev_status, const int* row_idx, const int* n_rows) {
  const long long big_tiles = (long long)((J + 127) / 128) * ((D + 127) / 128);
  if (big_tiles >= 148) {
    dim3 grid((D + 127) / 128, (J + 127) / 128);
    static PerDeviceOnce attr_once;   // function attributes are per device
    if (attr_once.first()) {
      cudaFuncSetAttribute(sgemm_pipe_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE * PIPE_STAGE_FLOATS * 4);
    }
    sgemm_pipe_kernel<0><<<grid, 256, PIPE * PIPE_STAGE_FLOATS * 4, s>>>(W, u, v, K, J, D, eta, dev_status, RowMap(), 0, 0,
                                                                         row_idx, n_rows);
  } else {
    dim3 grid((D + 63) / 64, (J + 63) / 64);
    apply_f32_kernel<1, 1><<<grid, 256, 0, s>>>(W, u, v, K, J, D, eta, dev_status);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

// Forward contraction through transposed copies of its operands (workspace: xt [D][ldk], wt [D][ldj] floats with
// ldk, ldj = K, J rounded up to 4): two bandwidth-bound transposing passes, then the pipelined kernel above, which
// runs faster than the kernel that transposes through registers.  src: the operand rows a_i (X rows, or pair
// differences already written as the factor v); copy: optional second destination of those rows (v = x).
long long forward_f32_nn_workspace_floats(int K, int J, int D) {
  return (long long)D * (((K + 3) & ~3) + ((J + 3) & ~3));
}

int launch_forward_f32_nn(cudaStream_t s, const float* W, RowMap src, RowMap copy, int K, int J, int D, float* ws,
                          RowMap z, RowMap part, long long split_stride, int max_splits, int* nsplit_out) {
  const int ldk = (K + 3) & ~3, ldj = (J + 3) & ~3;
  float* xt = ws;
  float* wt = ws + (size_t)D * ldk;
  RowMap wrows;
  wrows.base = const_cast<char*>(reinterpret_cast<const char*>(W));
  wrows.worker_stride = 0; wrows.ld = D; wrows.B = J > 0 ? J : 1; wrows.es = 4;
  const bool vec = (D & 3) == 0 && (src.ld & 3) == 0 && (reinterpret_cast<uintptr_t>(src.base) & 15) == 0 &&
                   (src.worker_stride & 15) == 0 && (reinterpret_cast<uintptr_t>(W) & 15) == 0 &&
                   (copy.base == nullptr || ((copy.ld & 3) == 0 && (reinterpret_cast<uintptr_t>(copy.base) & 15) == 0 &&
                                             (copy.worker_stride & 15) == 0));
  int transposes = 2;
  if (vec) {   // both operands in one launch
    TransposeJob jx, jw;
    jx.src = src; jx.dst = xt; jx.R = K; jx.C = D; jx.ldr = ldk; jx.copy = copy;
    jw.src = wrows; jw.dst = wt; jw.R = J; jw.C = D; jw.ldr = ldj; jw.copy = RowMap();
    const int ry = ((ldk > ldj ? ldk : ldj) + 63) / 64;
    transpose_rows_vec_kernel<<<dim3((D + 63) / 64, ry, 2), 256, 0, s>>>(jx, jw);
    transposes = 1;
  } else {
    transpose_rows_kernel<<<dim3((D + 31) / 32, (ldk + 31) / 32), 256, 0, s>>>(src, xt, K, D, ldk, copy);
    transpose_rows_kernel<<<dim3((D + 31) / 32, (ldj + 31) / 32), 256, 0, s>>>(wrows, wt, J, D, ldj, RowMap());
  }
  int ks = (part.base != nullptr && nsplit_out != nullptr) ? forward_f32_splits(K, J, D) : 1;
  if (ks > max_splits) ks = max_splits;
  if (nsplit_out != nullptr) *nsplit_out = ks;
  const int per = ((D + ks - 1) / ks + BK - 1) / BK * BK;
  RowMap a, b;
  a.base = reinterpret_cast<char*>(xt); a.worker_stride = 0; a.ld = ldk; a.B = D; a.es = 4;
  b.base = reinterpret_cast<char*>(wt); b.worker_stride = 0; b.ld = ldj; b.B = D; b.es = 4;
  static PerDeviceOnce attr_once;   // function attributes are per device
  if (attr_once.first())
    cudaFuncSetAttribute(sgemm_pipe_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, PIPE * PIPE_STAGE_FLOATS * 4);
  // rows of the output tile = samples (M = K), columns = classes (N = J), reduction over the D features
  dim3 grid((J + 127) / 128, (K + 127) / 128, ks);
  sgemm_pipe_kernel<1><<<grid, 256, PIPE * PIPE_STAGE_FLOATS * 4, s>>>(nullptr, a, b, D, K, ldj, 0.f, nullptr,
                                                                       ks > 1 ? part : z, per, split_stride, nullptr, nullptr);
  return cudaGetLastError() == cudaSuccess ? transposes + 1 : SFB_ERR_CUDA;
}

}  // namespace sfb
