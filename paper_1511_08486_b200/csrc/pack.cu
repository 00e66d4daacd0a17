// SF buffer bookkeeping: header and directory, CSR code streams, header validation.
// The buffer is the message the P workers would broadcast at commit() (Section 4.2); the layout is
// the wire format documented in include/sfb.h.  Integer offset arithmetic and copies only.
#include "common.cuh"

namespace sfb {
namespace {

struct HeaderImage {   // exactly the first 68 bytes of the 128-byte header
  uint32_t magic;
  uint16_t version;
  uint8_t model, dtype;
  uint32_t flags, P, B, J, D, clock, ldu, ldv;
  uint64_t stream_stride, total_bytes, streams_off;
  uint32_t cap_p;
};
static_assert(sizeof(HeaderImage) == 72, "header image is 68 bytes of fields plus 4 of tail padding");

__host__ HeaderImage make_header(const sfb_desc& d, const Layout& l, uint32_t clock) {
  HeaderImage h;
  h.magic = 0x31424653u;
  h.version = 1;
  h.model = (uint8_t)d.model;
  h.dtype = (l.es == 2) ? 1 : 0;
  h.flags = d.v_sparse ? 1u : 0u;
  h.P = d.P; h.B = d.B; h.J = d.J; h.D = d.D;
  h.clock = clock;
  h.ldu = l.ldu; h.ldv = l.ldv;
  h.stream_stride = (uint64_t)l.stream_stride;
  h.total_bytes = (uint64_t)l.total_bytes;
  h.streams_off = (uint64_t)l.streams_off;
  h.cap_p = (uint32_t)l.cap_p;
  return h;
}

// One block: thread t < 32 writes header word t (128 bytes); then threads stride over the directory.
__global__ void write_header_kernel(char* buf, HeaderImage h, long long u_bytes, const uint32_t* __restrict__ rowptr) {
  uint32_t* w = reinterpret_cast<uint32_t*>(buf);
  const uint32_t* src = reinterpret_cast<const uint32_t*>(&h);
  if (threadIdx.x < 32) w[threadIdx.x] = (threadIdx.x < 17) ? src[threadIdx.x] : 0u;
  const int dir_words = (int)((h.streams_off - 128) / 4);
  for (int t = threadIdx.x; t < dir_words; t += blockDim.x) {
    const int p = t >> 3, f = t & 7;
    uint32_t val = 0u;
    if (p < (int)h.P) {
      const uint64_t u_off = h.streams_off + (uint64_t)p * h.stream_stride;
      const uint64_t v_off = u_off + (uint64_t)u_bytes;
      switch (f) {
        case 0: val = (uint32_t)p; break;
        case 1: val = h.B; break;
        case 2: val = h.clock; break;
        case 3:
          if (rowptr != nullptr) {
            const uint32_t n = rowptr[(p + 1) * h.B] - rowptr[p * h.B];
            val = n < h.cap_p ? n : h.cap_p;
          } else if (h.flags & 1u) {   // no global row pointers: the count the worker's own stream carries
            val = reinterpret_cast<const uint32_t*>(buf + v_off)[h.B];
          }
          break;
        case 4: val = (uint32_t)(u_off & 0xffffffffu); break;
        case 5: val = (uint32_t)(u_off >> 32); break;
        case 6: val = (uint32_t)(v_off & 0xffffffffu); break;
        default: val = (uint32_t)(v_off >> 32); break;
      }
    }
    w[32 + t] = val;
  }
}

__global__ void check_header_kernel(const char* buf, HeaderImage h, int* dev_status) {
  const uint32_t* w = reinterpret_cast<const uint32_t*>(buf);
  const uint32_t* ref = reinterpret_cast<const uint32_t*>(&h);
  const int t = threadIdx.x;   // 32 threads
  bool ok = true;
  if (t < 17 && t != 7) ok = (w[t] == ref[t]);   // word 7 is the clock: any value is accepted
  if (t == 2) ok = ((w[t] & ~2u) == ref[t]);      // flag bit 1 (compacted) may be set or not
  if (!__all_sync(0xffffffffu, ok) && t == 0) atomicOr(dev_status, SFB_DEV_BAD_HEADER);
}

// grid.x = P workers; each block copies its worker's CSR rows into the stream.
__global__ void __launch_bounds__(256) pack_csr_kernel(char* buf, long long streams_off, long long stream_stride,
                                                       long long u_bytes, long long rp_bytes, long long idx_bytes,
                                                       int B, int cap_p, int D, const uint32_t* __restrict__ rowptr,
                                                       const uint32_t* __restrict__ idx, const float* __restrict__ val,
                                                       int* dev_status) {
  const int p = blockIdx.x;
  const int part = blockIdx.y, parts = gridDim.y;   // the worker's words are spread over gridDim.y blocks
  char* vb = buf + streams_off + (long long)p * stream_stride + u_bytes;
  uint32_t* rp = reinterpret_cast<uint32_t*>(vb);
  uint32_t* ix = reinterpret_cast<uint32_t*>(vb + rp_bytes);
  float* vl = reinterpret_cast<float*>(vb + rp_bytes + idx_bytes);
  const uint32_t base = rowptr[(size_t)p * B];
  const uint32_t nnz_true = rowptr[(size_t)(p + 1) * B] - base;
  const uint32_t nnz = nnz_true < (uint32_t)cap_p ? nnz_true : (uint32_t)cap_p;
  if (nnz_true > (uint32_t)cap_p && threadIdx.x == 0 && part == 0) atomicOr(dev_status, SFB_DEV_CAPACITY);
  const int rp_words = (int)(rp_bytes / 4);
  for (int t = part * blockDim.x + threadIdx.x; t < rp_words; t += parts * blockDim.x) {
    uint32_t r = 0u;
    if (t <= B) {
      r = rowptr[(size_t)p * B + t] - base;
      if (r > nnz) r = nnz;
    }
    rp[t] = r;
  }
  const int idx_words = (int)(idx_bytes / 4);
  bool bad = false;
  for (int t = part * blockDim.x + threadIdx.x; t < idx_words; t += parts * blockDim.x) {
    uint32_t c = 0u;
    float a = 0.f;
    if ((uint32_t)t < nnz) {
      c = idx[base + t];
      a = val[base + t];
      if (c >= (uint32_t)D) bad = true;
    }
    ix[t] = c;
    vl[t] = a;   // val block is padded to the same number of 4-byte words (fp32 values)
  }
  if (bad) atomicOr(dev_status, SFB_DEV_BAD_INDEX);
}

}  // namespace

int launch_write_header(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, uint32_t clock,
                        const uint32_t* rowptr) {
  write_header_kernel<<<1, 256, 0, s>>>(reinterpret_cast<char*>(sf_buf), make_header(d, l, clock), l.u_bytes, rowptr);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_check_header(cudaStream_t s, const void* sf_buf, const sfb_desc& d, const Layout& l, int* dev_status) {
  check_header_kernel<<<1, 32, 0, s>>>(reinterpret_cast<const char*>(sf_buf), make_header(d, l, 0), dev_status);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

int launch_pack_csr(cudaStream_t s, void* sf_buf, const sfb_desc& d, const Layout& l, const uint32_t* rowptr,
                    const uint32_t* idx, const float* val, int* dev_status) {
  const int parts = (l.cap_p + 2047) / 2048 < 1 ? 1 : ((l.cap_p + 2047) / 2048 > 64 ? 64 : (l.cap_p + 2047) / 2048);
  pack_csr_kernel<<<dim3(d.P, parts), 256, 0, s>>>(reinterpret_cast<char*>(sf_buf), l.streams_off, l.stream_stride, l.u_bytes,
                                      l.rp_bytes, l.idx_bytes, d.B, l.cap_p, d.D, rowptr, idx, val, dev_status);
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

}  // namespace sfb
