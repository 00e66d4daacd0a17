// Operand splitting for the error-compensated tf32 kernels (SFB_PATH_TF32X3).
//
// The tensor core sees only the top 10 mantissa bits of an fp32 operand: x = hi + lo with hi = x with its low 13
// mantissa bits cleared and lo = x - hi, exact in fp32.  A product a b is then hi(a) hi(b), which the tf32
// instruction computes from the fp32 operands as they are, plus the corrections lo(a) b + a lo(b) (lo lo, about
// 2^-22 of the product, is dropped).  The corrections are 2^-10 of the product, so bf16 operands carry them to
// 2^-18: the kernels here write, for every fp32 operand matrix, a bf16 "correction operand" of twice the
// reduction length whose product with the other side's correction operand is exactly that sum:
//
//     A side:  [ lo(a) | a ]        B side:  [ b | lo(b) ]        (both halves rounded to nearest bf16)
//
// 32 reduction steps of the fp32 operand (one 128-byte atom) become 64 bf16 steps (again 128 bytes), so the
// correction operand has the size and the tiling of the fp32 one and the GEMM kernel loads it with the same
// coordinates.
//
// Two layouts, as the GEMM's operands have:
//   K-major (forward: sample rows and W rows, reduction along the row): dst[row][atom][64], the atom's 32
//     remainders and its 32 values side by side.
//   MN-major (apply: factor rows, reduction over the pairs): per reduction block of 32 pairs, 64 lines of
//     ldc values: dst[block][64][ldc], the 32 remainder lines and the 32 value lines.
#include "common.cuh"

namespace sfb {
namespace {

__device__ __forceinline__ float remainder_tf32(float x) {
  return x - __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  const __nv_bfloat162 p = __floats2bfloat162_rn(a, b);   // a in the low half = the lower address
  return *reinterpret_cast<const uint32_t*>(&p);
}

// values and remainders of eight consecutive fp32 values -> two 16-byte units
__device__ __forceinline__ void split8(const float4& x0, const float4& x1, uint4& val, uint4& rem) {
  val = make_uint4(pack_bf16(x0.x, x0.y), pack_bf16(x0.z, x0.w), pack_bf16(x1.x, x1.y), pack_bf16(x1.z, x1.w));
  rem = make_uint4(pack_bf16(remainder_tf32(x0.x), remainder_tf32(x0.y)), pack_bf16(remainder_tf32(x0.z), remainder_tf32(x0.w)),
                   pack_bf16(remainder_tf32(x1.x), remainder_tf32(x1.y)), pack_bf16(remainder_tf32(x1.z), remainder_tf32(x1.w)));
}

// K-major.  One thread per (row, 8 values); cols is a multiple of 4, rows are 16-byte aligned.
__global__ void __launch_bounds__(256) split_k_kernel(RowMap src, int rows, int cols, int atoms, uint4* __restrict__ dst,
                                                      int a_side) {
  const long long t = (long long)blockIdx.x * 256 + threadIdx.x;
  const int per_row = atoms * 4;
  const long long row = t / per_row;
  if (row >= rows) return;
  const int g = (int)(t - row * per_row);   // group of 8 values inside the row
  const float* x = reinterpret_cast<const float*>(src.row((int)row)) + g * 8;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  const float4 x0 = (g * 8 < cols) ? __ldg(reinterpret_cast<const float4*>(x)) : zero;
  const float4 x1 = (g * 8 + 4 < cols) ? __ldg(reinterpret_cast<const float4*>(x) + 1) : zero;
  uint4 val, rem;
  split8(x0, x1, val, rem);
  // atom g / 4 of the row: eight 16-byte units, the first four of one kind and the last four of the other
  uint4* atom = dst + (row * atoms + (g >> 2)) * 8;
  const int q = g & 3;
  atom[q] = a_side ? rem : val;
  atom[4 + q] = a_side ? val : rem;
}

// MN-major.  grid = (reduction blocks, groups of 8 units of 8 values along the padded row); block = 32 lines x 8 units.
__global__ void __launch_bounds__(256) split_mn_kernel(RowMap src, int cols, int workers, int k_bb, int k_wp, int k_bpw,
                                                       uint4* __restrict__ dst, int ldc, int a_side) {
  const int unit = blockIdx.y * 8 + (threadIdx.x & 7);   // 8 values = 16 bytes of bf16
  const int line = threadIdx.x >> 3;                      // 0..31: pair inside the reduction block
  const int blk = blockIdx.x;
  if (unit * 8 >= ldc) return;
  int worker, row;
  if (k_wp == 1) { worker = blk / k_bpw; row = (blk % k_bpw) * 32 + line; }        // 32 rows of one worker
  else { worker = blk * k_wp + line / k_bb; row = line % k_bb; }                  // k_bb rows of each of k_wp workers
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 x0 = zero, x1 = zero;
  if (worker < workers && row < src.B) {
    const float* x = reinterpret_cast<const float*>(src.row(worker * src.B + row)) + unit * 8;
    if (unit * 8 < cols) x0 = __ldg(reinterpret_cast<const float4*>(x));
    if (unit * 8 + 4 < cols) x1 = __ldg(reinterpret_cast<const float4*>(x) + 1);
  }
  uint4 val, rem;
  split8(x0, x1, val, rem);
  const size_t units_per_line = (size_t)ldc / 8;
  uint4* base = dst + ((size_t)blk * 64) * units_per_line + unit;
  base[(size_t)(a_side ? line : 32 + line) * units_per_line] = rem;
  base[(size_t)(a_side ? 32 + line : line) * units_per_line] = val;
}

}  // namespace

int launch_split_k(cudaStream_t s, RowMap src, int rows, int cols, void* dst, bool a_side) {
  if (rows <= 0) return 0;
  const int atoms = (cols + 31) / 32;
  const long long threads = (long long)rows * atoms * 4;
  split_k_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, s>>>(src, rows, cols, atoms, reinterpret_cast<uint4*>(dst),
                                                                  a_side ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_split_mn(cudaStream_t s, RowMap src, int cols, int workers, int k_bb, int k_wp, int k_bpw, int blocks,
                    void* dst, int ldc, bool a_side) {
  if (blocks <= 0) return 0;
  const dim3 grid((unsigned)blocks, (unsigned)((ldc / 8 + 7) / 8));
  split_mn_kernel<<<grid, 256, 0, s>>>(src, cols, workers, k_bb, k_wp, k_bpw, reinterpret_cast<uint4*>(dst), ldc,
                                       a_side ? 1 : 0);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

}  // namespace sfb
