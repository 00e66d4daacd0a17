// Host side of the C ABI declared in include/sfb.h: argument checks, workspace, kernel sequencing.
// Every step of the path runs in the CUDA kernels of this library; there is no CPU fallback.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"
#include "umma_api.cuh"

using namespace sfb;

struct sfb_ctx {
  sfb_desc d;
  Layout l;
  cudaStream_t stream;
  int K;
  int* dev_status;          // sticky device status word
  float* wt_ws;             // SC, fp32 path: atom-major copy of W for the forward
  float* a_dense;           // SC, tf32 path: dense rows of the codes, [K][ldv]
  void* csc_ws;             // SC, fp32 path: scratch of the atom-major re-sort of the codes (when K fits)
  // sfb_step: work that does not depend on the factors (codes into the buffer, header, atom-major re-sort of
  // the codes) runs on this stream beside the forward pass, forked and joined by events
  cudaStream_t aux;
  cudaEvent_t aux_fork, aux_join;
  bool aux_ok;
  float* f32_part;          // fp32 dense path: partial products [splits][K][ldp] of a split forward reduction
  int ldp, f32_splits;
  // DML, fp32 path: which pairs of the current step contribute (u_i != 0), their ordered list and its length;
  // the step's apply leaves the others out (bit-identical result, fewer multiply-adds)
  uint8_t* dml_active;
  int* dml_idx;             // [K] indices followed by the count
  int last_step_K;          // K of the last sfb_step (0: none yet) and whether its apply walked the list
  bool last_step_listed;
  void* compact_ws;         // compact = 1: flags, new slots and per-worker counts of the pair compaction
  int* kept_idx;            // compact = 1, fp32 path: ordered list of the kept pairs' slots, followed by its length
  float* f32_nn_ws;         // fp32 dense path: transposed copies of the forward's operands (large shapes only)
  float* loss_rows;         // sfb_loss: fp32 products [K][ldl], allocated by the first call
  float* loss_i;            // sfb_loss: per-sample objective [K]
  // sfb_step_host: two sets of device staging buffers for the step's host inputs (allocated on first
  // use), filled on a side stream so that the copy of step t+1 overlaps the kernels of step t
  char* host_stage[2][6];
  size_t host_stage_bytes[2][6];
  cudaStream_t copy_stream;
  cudaEvent_t copied[2], consumed[2];
  bool host_ready;
  uint64_t host_steps;
  // bf16 path: bf16 copy of W, refreshed by the apply.  Compensated tf32 path: W's correction operand
  // (bf16 [value | remainder] per 32 columns, as many bytes as W), rebuilt before a forward pass when stale.
  __nv_bfloat16* w_shadow;
  const void* shadow_of;    // W pointer the shadow currently mirrors (nullptr = stale)
  UmmaPlan* umma;           // tensor-core plan (tensor maps), TF32 / BF16 paths
  int64_t launches;
  bool profiling;
  int prof_n;                       // steps recorded since the last read
  cudaEvent_t prof_ev[128][3];      // start / after factors / after apply
  bool prof_have_events;
};

namespace {

bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_desc(const sfb_desc* d) {
  if (d == nullptr) return SFB_ERR_ARG;
  if (d->model < SFB_MLR || d->model > SFB_SC) return SFB_ERR_ARG;
  if (d->path < SFB_PATH_F32 || d->path > SFB_PATH_TF32X3) return SFB_ERR_ARG;
  if (d->J <= 0 || d->D <= 0 || d->P <= 0 || d->B <= 0) return SFB_ERR_SHAPE;
  if ((long long)d->P * d->B > (1 << 24)) return SFB_ERR_SHAPE;
  if (d->model == SFB_SC) {
    if (!d->v_sparse) return SFB_ERR_UNSUPPORTED;          // dictionary updates take CSR codes
    if (d->path == SFB_PATH_BF16) return SFB_ERR_UNSUPPORTED;   // fp32 sparse path, or dense tf32 on tensor cores
    if (d->nnz_capacity == 0 || d->nnz_capacity % (32ull * d->P) != 0) return SFB_ERR_SHAPE;
    if (d->nnz_capacity / d->P > (1ull << 30)) return SFB_ERR_SHAPE;
  } else if (d->v_sparse) {
    return SFB_ERR_UNSUPPORTED;
  }
  if (d->path == SFB_PATH_BF16 && d->model != SFB_MLR) return SFB_ERR_UNSUPPORTED;
  if (d->path == SFB_PATH_BF16 && (d->D % 8) != 0) return SFB_ERR_SHAPE;   // 16-byte rows of bf16 X and W shadow
  if ((d->path == SFB_PATH_TF32 || d->path == SFB_PATH_TF32X3) && (d->D % 4) != 0)
    return SFB_ERR_SHAPE;   // 16-byte rows of fp32 X and W
  if (d->model == SFB_DML && !(d->margin > 0.f)) return SFB_ERR_ARG;
  if (d->compact != 0 && d->compact != 1) return SFB_ERR_ARG;
  if (d->compact && d->v_sparse) return SFB_ERR_UNSUPPORTED;   // pair compaction is defined for dense v
  return SFB_OK;
}

RowMap caller_rows(const void* base, int ld, int B, int es) {
  RowMap m;
  m.base = const_cast<char*>(reinterpret_cast<const char*>(base));
  m.worker_stride = (long long)B * ld * es;
  m.ld = ld; m.B = B; m.es = es;
  return m;
}
RowMap stream_u(const sfb_ctx* c, const void* sf_buf) {
  RowMap m;
  m.base = const_cast<char*>(reinterpret_cast<const char*>(sf_buf)) + c->l.streams_off;
  m.worker_stride = c->l.stream_stride;
  m.ld = c->l.ldu; m.B = c->d.B; m.es = c->l.es;
  return m;
}
RowMap stream_v(const sfb_ctx* c, const void* sf_buf) {
  RowMap m = stream_u(c, sf_buf);
  m.base += c->l.u_bytes;
  m.ld = c->l.ldv;
  return m;
}
RowMap dense_codes(const sfb_ctx* c) { return caller_rows(c->a_dense, c->l.ldv, c->d.B, 4); }

// cap_p > 0: every worker's rows end after its first cap_p nonzeros, as in the stream pack_csr writes
CsrView global_codes(const sfb_aux* a, int B, int cap_p = 0) {
  CsrView v;
  memset(&v, 0, sizeof(v));
  v.rowptr = a->rowptr; v.idx = a->idx; v.val = reinterpret_cast<const float*>(a->val); v.B = B;
  v.cap_p = cap_p;
  return v;
}
CsrView stream_codes(const sfb_ctx* c, const void* sf_buf) {
  CsrView v;
  memset(&v, 0, sizeof(v));
  v.base = reinterpret_cast<const char*>(sf_buf);
  v.streams_off = c->l.streams_off; v.stream_stride = c->l.stream_stride; v.v_off = c->l.u_bytes;
  v.rp_bytes = c->l.rp_bytes; v.idx_bytes = c->l.idx_bytes; v.B = c->d.B;
  return v;
}

int check_aux(const sfb_ctx* c, const sfb_aux* a) {
  if (a == nullptr) return SFB_ERR_ARG;
  switch (c->d.model) {
    case SFB_MLR:
      if (a->labels == nullptr || !aligned(a->labels, 4)) return SFB_ERR_ARG;
      if (a->dual != nullptr && (!aligned(a->dual, 16) || !(a->sdca_step > 0.f && a->sdca_step <= 1.f))) return SFB_ERR_ARG;
      return SFB_OK;
    case SFB_DML: return (a->Xb != nullptr && a->similar != nullptr && aligned(a->Xb, 16)) ? SFB_OK : SFB_ERR_ARG;
    default:
      return (a->rowptr && a->idx && a->val && a->Xdata && aligned(a->rowptr, 4) && aligned(a->idx, 4) &&
              aligned(a->val, 4) && aligned(a->Xdata, 4)) ? SFB_OK : SFB_ERR_ARG;
  }
}

#define ACC(expr)                  \
  do {                             \
    const int r_ = (expr);         \
    if (r_ < 0) return r_;         \
    c->launches += r_;             \
  } while (0)

bool has_shadow(const sfb_ctx* c) { return c->d.path == SFB_PATH_BF16 || c->d.path == SFB_PATH_TF32X3; }

// Refreshes the shadow of W (bf16 copy, or correction operand) if it does not mirror this W.
int ensure_shadow(sfb_ctx* c, const void* W) {
  if (!has_shadow(c) || c->shadow_of == W) return SFB_OK;
  if (c->d.path == SFB_PATH_BF16) {
    ACC(launch_cast_bf16(c->stream, reinterpret_cast<const float*>(W), c->w_shadow, (long long)c->d.J * c->d.D));
  } else {
    RowMap w;
    w.base = const_cast<char*>(reinterpret_cast<const char*>(W));
    w.ld = c->d.D; w.B = c->d.J; w.es = 4; w.worker_stride = 0;
    ACC(launch_split_k(c->stream, w, c->d.J, c->d.D, c->w_shadow, false));
  }
  c->shadow_of = W;
  return SFB_OK;
}

// Factors of one minibatch written through the row maps u / v (v.base == nullptr: v not wanted).
// workers > 0: the minibatch holds only that many workers' samples and u / v / codes start at the first of them.
// for_apply: the apply of exactly these rows (all K pairs, no compaction in between) follows in the same call, so
// the compensated path may write the apply's correction operands while it writes the factors.
int factors_into(sfb_ctx* c, const void* W, const void* X, const sfb_aux* aux, RowMap u, RowMap v, CsrView codes,
                 int workers = 0, bool for_apply = false) {
  const sfb_desc& d = c->d;
  const int K = workers > 0 ? workers * d.B : c->K;
  const float* Wf = reinterpret_cast<const float*>(W);
  if (d.model == SFB_SC && d.path == SFB_PATH_F32) {
    ACC(launch_sc_forward_ws(c->stream, Wf, c->wt_ws, codes, reinterpret_cast<const float*>(aux->Xdata), u, K, d.J,
                             d.D, c->dev_status));
    return SFB_OK;
  }
  if (d.model == SFB_SC) {   // dense alternative: the codes as dense tf32 rows through the tensor-core GEMM
    const RowMap a = dense_codes(c);
    // plain tf32: the code values are rounded to nearest tf32 as they are densified; the compensated path keeps
    // them exact (its kernels split every operand into what the tensor core sees and the rest)
    // compensated path: the same kernel writes the rows' correction operands (when a row fits in shared memory)
    const bool with_corr = d.path == SFB_PATH_TF32X3 && workers == 0 && densify_corr_fits(a.ld);
    const CorrOut a_corr = with_corr ? umma_codes_corr(c->umma, for_apply) : CorrOut();
    if (with_corr) ACC(launch_densify_codes_corr(c->stream, codes, a, K, d.D, c->dev_status, a_corr));
    else ACC(launch_densify_codes(c->stream, codes, a, K, d.D, c->dev_status, d.path == SFB_PATH_TF32));
    {
      const int r = ensure_shadow(c, W);
      if (r < 0) return r;
    }
    ACC(umma_forward_sc(c->umma, c->stream, W, a, u, reinterpret_cast<const float*>(aux->Xdata), c->dev_status, workers,
                        c->w_shadow, for_apply, with_corr ? &a_corr : nullptr));
    return SFB_OK;
  }
  if (d.path == SFB_PATH_F32) {
    const float* Xb = (d.model == SFB_DML) ? reinterpret_cast<const float*>(aux->Xb) : nullptr;
    // partial products of a split reduction live in the context's workspace, laid out like caller rows
    const RowMap part = caller_rows(c->f32_part, c->ldp, d.B, 4);
    const long long sstride = (long long)c->K * c->ldp * 4;
    int ks = 1;
    if (c->f32_nn_ws != nullptr && (Xb == nullptr || v.base != nullptr)) {
      RowMap src = caller_rows(X, d.D, d.B, 4), copy = v;
      if (Xb != nullptr) {   // pair differences first (they are the factor v), then contracted from there
        ACC(launch_diff_rows(c->stream, reinterpret_cast<const float*>(X), Xb, v, K, d.D));
        src = v;
        copy = RowMap();
      }
      ACC(launch_forward_f32_nn(c->stream, Wf, src, copy, K, d.J, d.D, c->f32_nn_ws, u, part, sstride, c->f32_splits,
                                &ks));
    } else {
      ACC(launch_forward_f32(c->stream, Wf, reinterpret_cast<const float*>(X), Xb, K, d.J, d.D, u, v, part, sstride,
                             c->f32_splits, &ks));
    }
    const RowMap zsrc = ks > 1 ? part : u;
    if (d.model == SFB_MLR)
      ACC(launch_finish_mlr(c->stream, zsrc, u, aux->labels, K, d.J, c->dev_status, ks, sstride,
                            reinterpret_cast<float*>(aux->dual), aux->sdca_step));
    else ACC(launch_finish_dml(c->stream, zsrc, u, aux->similar, d.margin, K, d.J, ks, sstride, c->dml_active));
    return SFB_OK;
  }
  // tensor-core paths
  {
    const int r = ensure_shadow(c, W);
    if (r < 0) return r;
  }
  ACC(umma_forward(c->umma, c->stream, W, c->w_shadow, X, aux, u, v, c->dev_status, workers, for_apply));
  return SFB_OK;
}

}  // namespace

extern "C" {

const char* sfb_strerror(int code) {
  switch (code) {
    case SFB_OK: return "ok";
    case SFB_ERR_ARG: return "bad argument (null or misaligned pointer, bad enum, K not a whole number of worker streams)";
    case SFB_ERR_SHAPE: return "unsupported sizes";
    case SFB_ERR_UNSUPPORTED: return "model/path combination not provided, or not an sm_100 device";
    case SFB_ERR_CUDA: return "a CUDA call failed";
    case SFB_ERR_ALLOC: return "workspace allocation failed";
    case SFB_ERR_SCRATCH: return "problem exceeds the fixed scratch array of the no-allocation entry point";
    default: return "unknown error";
  }
}

size_t sfb_sf_buffer_bytes(const sfb_desc* desc) {
  if (check_desc(desc) != SFB_OK) return 0;
  return (size_t)make_layout(*desc).total_bytes;
}

int sfb_sf_buffer_layout(const sfb_desc* desc, uint64_t* streams_off, uint64_t* stream_stride) {
  if (streams_off == nullptr || stream_stride == nullptr) return SFB_ERR_ARG;
  const int r = check_desc(desc);
  if (r != SFB_OK) return r;
  const Layout l = make_layout(*desc);
  *streams_off = (uint64_t)l.streams_off;
  *stream_stride = (uint64_t)l.stream_stride;
  return SFB_OK;
}

int sfb_ld(const sfb_desc* desc, int32_t* ldu, int32_t* ldv) {
  const int r = check_desc(desc);
  if (r != SFB_OK) return r;
  const Layout l = make_layout(*desc);
  if (ldu) *ldu = l.ldu;
  if (ldv) *ldv = l.ldv;
  return SFB_OK;
}

int sfb_create(const sfb_desc* desc, void* cuda_stream, sfb_ctx** out) {
  if (out == nullptr) return SFB_ERR_ARG;
  *out = nullptr;
  const int r = check_desc(desc);
  if (r != SFB_OK) return r;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SFB_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SFB_ERR_CUDA;
  if (major != 10) return SFB_ERR_UNSUPPORTED;   // kernels are built for sm_100a only
  sfb_ctx* c = new (std::nothrow) sfb_ctx();
  if (c == nullptr) return SFB_ERR_ALLOC;
  memset(c, 0, sizeof(*c));
  c->d = *desc;
  c->l = make_layout(*desc);
  c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  c->K = desc->P * desc->B;
  bool ok = cudaMalloc(&c->dev_status, 256) == cudaSuccess;
  if (ok) ok = cudaMemsetAsync(c->dev_status, 0, 256, c->stream) == cudaSuccess;
  if (ok && desc->model == SFB_SC && desc->path == SFB_PATH_F32)
    ok = cudaMalloc(&c->wt_ws, (size_t)sc_forward_workspace_bytes(desc->J, desc->D)) == cudaSuccess;
  if (ok && desc->model == SFB_SC && desc->path == SFB_PATH_F32 && sc_csc_supported(c->K))
    ok = cudaMalloc(&c->csc_ws, (size_t)sc_csc_workspace_bytes(c->K, desc->D, (long long)desc->nnz_capacity)) == cudaSuccess;
  if (ok && desc->model == SFB_SC && (desc->path == SFB_PATH_TF32 || desc->path == SFB_PATH_TF32X3))
    ok = cudaMalloc(&c->a_dense, (size_t)c->K * c->l.ldv * 4) == cudaSuccess;
  if (ok && desc->model != SFB_SC && desc->path == SFB_PATH_F32) {
    const int ks = forward_f32_splits(c->K, desc->J, desc->D);
    c->ldp = (desc->J + 3) & ~3;
    c->f32_splits = ks;
    if (ks > 1) ok = cudaMalloc(&c->f32_part, (size_t)ks * c->K * c->ldp * 4) == cudaSuccess;
    if (ok && desc->model == SFB_DML) {
      ok = cudaMalloc(&c->dml_active, (size_t)c->K) == cudaSuccess;
      if (ok) ok = cudaMalloc(&c->dml_idx, ((size_t)c->K + 1) * 4) == cudaSuccess;
    }
    // shapes with at least a tile of work per dimension take the forward through transposed operand copies
    const long long nn_floats = forward_f32_nn_workspace_floats(c->K, desc->J, desc->D);
    if (ok && c->K >= 128 && desc->J >= 64 && desc->D >= 512 && nn_floats * 4 <= (2LL << 30))
      ok = cudaMalloc(&c->f32_nn_ws, (size_t)nn_floats * 4) == cudaSuccess;
  }
  if (ok) {
    if (cudaStreamCreateWithFlags(&c->aux, cudaStreamNonBlocking) == cudaSuccess) {
      const bool e1 = cudaEventCreateWithFlags(&c->aux_fork, cudaEventDisableTiming) == cudaSuccess;
      const bool e2 = e1 && cudaEventCreateWithFlags(&c->aux_join, cudaEventDisableTiming) == cudaSuccess;
      c->aux_ok = e2;
      if (!e2) {
        if (e1) cudaEventDestroy(c->aux_fork);
        cudaStreamDestroy(c->aux);
        cudaGetLastError();
      }
    }
  }
  if (ok && desc->path == SFB_PATH_BF16) ok = cudaMalloc(&c->w_shadow, (size_t)desc->J * desc->D * 2) == cudaSuccess;
  if (ok && desc->path == SFB_PATH_TF32X3)
    ok = cudaMalloc(&c->w_shadow, (size_t)desc->J * ((desc->D + 31) / 32) * 128) == cudaSuccess &&
         // columns beyond D inside the last atom are zeros for good: nothing writes them again
         cudaMemset(c->w_shadow, 0, (size_t)desc->J * ((desc->D + 31) / 32) * 128) == cudaSuccess;
  if (ok && desc->compact) {
    ok = cudaMalloc(&c->compact_ws, (size_t)compact_workspace_bytes(c->K, desc->P)) == cudaSuccess;
    if (ok && desc->path == SFB_PATH_F32) ok = cudaMalloc(&c->kept_idx, ((size_t)c->K + 1) * 4) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    sfb_destroy(c);
    return SFB_ERR_ALLOC;
  }
  if (desc->path != SFB_PATH_F32) {
    const int ur = umma_plan_create(c->d, c->l, &c->umma);
    if (ur != SFB_OK) {
      sfb_destroy(c);
      return ur;
    }
  }
  *out = c;
  return SFB_OK;
}

int sfb_destroy(sfb_ctx* c) {
  if (c == nullptr) return SFB_ERR_ARG;
  cudaStreamSynchronize(c->stream);
  if (c->aux_ok) {
    cudaStreamSynchronize(c->aux);
    cudaEventDestroy(c->aux_fork);
    cudaEventDestroy(c->aux_join);
    cudaStreamDestroy(c->aux);
  }
  if (c->umma) umma_plan_destroy(c->umma);
  if (c->prof_have_events)
    for (int i = 0; i < 128; ++i)
      for (int e = 0; e < 3; ++e) cudaEventDestroy(c->prof_ev[i][e]);
  if (c->dev_status) cudaFree(c->dev_status);
  if (c->wt_ws) cudaFree(c->wt_ws);
  if (c->a_dense) cudaFree(c->a_dense);
  if (c->csc_ws) cudaFree(c->csc_ws);
  if (c->f32_part) cudaFree(c->f32_part);
  if (c->f32_nn_ws) cudaFree(c->f32_nn_ws);
  if (c->compact_ws) cudaFree(c->compact_ws);
  if (c->kept_idx) cudaFree(c->kept_idx);
  if (c->dml_active) cudaFree(c->dml_active);
  if (c->dml_idx) cudaFree(c->dml_idx);
  if (c->loss_rows) cudaFree(c->loss_rows);
  if (c->loss_i) cudaFree(c->loss_i);
  for (int k = 0; k < 2; ++k)
    for (int i = 0; i < 6; ++i)
      if (c->host_stage[k][i]) cudaFree(c->host_stage[k][i]);
  if (c->host_ready) {
    cudaStreamSynchronize(c->copy_stream);
    for (int k = 0; k < 2; ++k) {
      cudaEventDestroy(c->copied[k]);
      cudaEventDestroy(c->consumed[k]);
    }
    cudaStreamDestroy(c->copy_stream);
  }
  if (c->w_shadow) cudaFree(c->w_shadow);
  delete c;
  return SFB_OK;
}

int sfb_prox(sfb_ctx* c, void* W) {
  if (c == nullptr || W == nullptr || !aligned(W, 16)) return SFB_ERR_ARG;
  if (c->d.model != SFB_SC) return SFB_OK;   // h = 0 for the MLR and DML workloads: identity
  ACC(launch_prox_unit_columns(c->stream, reinterpret_cast<float*>(W), c->d.J, c->d.D));
  c->shadow_of = nullptr;   // W changed
  return SFB_OK;
}

int sfb_loss(sfb_ctx* c, const void* W, const void* X, const sfb_aux* aux, double* loss) {
  if (c == nullptr || W == nullptr || loss == nullptr) return SFB_ERR_ARG;
  if (!aligned(W, 16) || !aligned(loss, 8)) return SFB_ERR_ARG;
  int r = check_aux(c, aux);
  if (r != SFB_OK) return r;
  const sfb_desc& d = c->d;
  if (d.model != SFB_SC && (X == nullptr || !aligned(X, 16))) return SFB_ERR_ARG;
  const int ldl = (d.J + 3) & ~3;
  if (c->loss_rows == nullptr) {
    bool ok = cudaMalloc(&c->loss_rows, (size_t)c->K * ldl * 4) == cudaSuccess;
    if (ok) ok = cudaMalloc(&c->loss_i, (size_t)c->K * 4) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      if (c->loss_rows) cudaFree(c->loss_rows);
      c->loss_rows = nullptr;
      return SFB_ERR_ALLOC;
    }
  }
  const RowMap rows = caller_rows(c->loss_rows, ldl, d.B, 4);
  const RowMap none = caller_rows(nullptr, c->l.ldv, d.B, c->l.es);
  if (d.model == SFB_SC) {
    // u_i = W a_i - x_i by the path's own forward (sparse gather, or dense tf32 rows)
    r = factors_into(c, W, X, aux, rows, none, global_codes(aux, d.B));
    if (r < 0) return r;
  } else if (d.path == SFB_PATH_F32 || d.model == SFB_DML) {
    const float* Xb = (d.model == SFB_DML) ? reinterpret_cast<const float*>(aux->Xb) : nullptr;
    ACC(launch_forward_f32(c->stream, reinterpret_cast<const float*>(W), reinterpret_cast<const float*>(X), Xb, c->K,
                           d.J, d.D, rows, none));
  } else {
    r = ensure_shadow(c, W);
    if (r < 0) return r;
    const bool bf16 = d.path == SFB_PATH_BF16;
    ACC(umma_forward_rows(c->umma, c->stream, bf16 ? (const void*)c->w_shadow : W, caller_rows(X, d.D, d.B, c->l.es),
                          rows, c->dev_status, nullptr, nullptr, nullptr, nullptr, 1, 0, 0, c->w_shadow));
  }
  ACC(launch_sample_loss(c->stream, d.model, rows, aux->labels, aux->similar, d.margin, c->K, d.J, c->loss_i, loss,
                         c->dev_status));
  return SFB_OK;
}

int sfb_active_pairs(sfb_ctx* c, int32_t* n) {
  if (c == nullptr || n == nullptr) return SFB_ERR_ARG;
  *n = 0;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  if (c->last_step_K == 0) return SFB_OK;
  if (c->d.compact) {   // the pair counts the compaction left in its workspace, over the workers the step applied
    const int workers = c->last_step_K / c->d.B;
    int32_t* h = new (std::nothrow) int32_t[workers];
    if (h == nullptr) return SFB_ERR_ALLOC;
    const char* counts = reinterpret_cast<const char*>(c->compact_ws) + pad_to(c->K, 256) + pad_to((long long)c->K * 4, 256);
    const bool ok = cudaMemcpy(h, counts, (size_t)workers * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    for (int p = 0; ok && p < workers; ++p) *n += h[p];
    delete[] h;
    return ok ? SFB_OK : SFB_ERR_CUDA;
  }
  if (c->dml_idx == nullptr || !c->last_step_listed) {
    *n = c->last_step_K;
    return SFB_OK;
  }
  int32_t h = 0;
  if (cudaMemcpy(&h, c->dml_idx + c->K, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return SFB_ERR_CUDA;
  *n = h;
  return SFB_OK;
}

int sfb_wire_bytes(sfb_ctx* c, const void* sf_buf, uint64_t* bytes) {
  if (c == nullptr || sf_buf == nullptr || bytes == nullptr) return SFB_ERR_ARG;
  *bytes = 0;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  const sfb_desc& d = c->d;
  uint32_t* dir = new (std::nothrow) uint32_t[(size_t)d.P * 8];
  if (dir == nullptr) return SFB_ERR_ALLOC;
  const bool ok = cudaMemcpy(dir, reinterpret_cast<const char*>(sf_buf) + 128, (size_t)d.P * 32, cudaMemcpyDeviceToHost) ==
                  cudaSuccess;
  uint64_t total = 128 + (uint64_t)d.P * 32;
  for (int p = 0; ok && p < d.P; ++p) {
    const uint64_t n_sf = dir[p * 8 + 1] < (uint32_t)d.B ? dir[p * 8 + 1] : (uint32_t)d.B, nnz = dir[p * 8 + 3];
    if (d.v_sparse) total += n_sf * d.J * c->l.es + ((uint64_t)d.B + 1) * 4 + nnz * (4 + (uint64_t)c->l.es);
    else total += n_sf * ((uint64_t)d.J + d.D) * c->l.es;
  }
  delete[] dir;
  if (!ok) return SFB_ERR_CUDA;
  *bytes = total;
  return SFB_OK;
}

int sfb_invalidate(sfb_ctx* c) {
  if (c == nullptr) return SFB_ERR_ARG;
  c->shadow_of = nullptr;
  return SFB_OK;
}

int64_t sfb_launch_count(const sfb_ctx* c) { return c ? c->launches : 0; }

int sfb_profile(sfb_ctx* c, int enable) {
  if (c == nullptr) return SFB_ERR_ARG;
  if (enable && !c->prof_have_events) {
    for (int i = 0; i < 128; ++i)
      for (int e = 0; e < 3; ++e)
        if (cudaEventCreate(&c->prof_ev[i][e]) != cudaSuccess) return SFB_ERR_CUDA;
    c->prof_have_events = true;
  }
  c->profiling = enable != 0;
  c->prof_n = 0;
  return SFB_OK;
}

int sfb_stage_ms(sfb_ctx* c, float* factors_ms, float* apply_ms, int32_t* steps) {
  if (c == nullptr || factors_ms == nullptr || apply_ms == nullptr || steps == nullptr) return SFB_ERR_ARG;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  const int n = c->prof_n < 128 ? c->prof_n : 128;
  float f = 0.f, a = 0.f;
  for (int i = 0; i < n; ++i) {
    float t0 = 0.f, t1 = 0.f;
    if (cudaEventElapsedTime(&t0, c->prof_ev[i][0], c->prof_ev[i][1]) != cudaSuccess) return SFB_ERR_CUDA;
    if (cudaEventElapsedTime(&t1, c->prof_ev[i][1], c->prof_ev[i][2]) != cudaSuccess) return SFB_ERR_CUDA;
    f += t0;
    a += t1;
  }
  *factors_ms = f; *apply_ms = a; *steps = n;
  c->prof_n = 0;
  return SFB_OK;
}

int sfb_status(sfb_ctx* c, int32_t* device_status) {
  if (c == nullptr || device_status == nullptr) return SFB_ERR_ARG;
  int32_t h = 0;
  if (cudaMemcpyAsync(&h, c->dev_status, 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  if (cudaMemsetAsync(c->dev_status, 0, 4, c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  *device_status = h;
  return SFB_OK;
}

int sfb_compute_factors(sfb_ctx* c, const void* W, const void* X, const sfb_aux* aux, void* U, void* V) {
  if (c == nullptr || W == nullptr || U == nullptr) return SFB_ERR_ARG;
  if (!aligned(W, 16) || !aligned(U, 16) || (V != nullptr && !aligned(V, 16))) return SFB_ERR_ARG;
  int r = check_aux(c, aux);
  if (r != SFB_OK) return r;
  if (c->d.model != SFB_SC && (X == nullptr || !aligned(X, 16))) return SFB_ERR_ARG;
  RowMap u = caller_rows(U, c->l.ldu, c->d.B, c->l.es);
  RowMap v = caller_rows(c->d.model == SFB_SC ? nullptr : V, c->l.ldv, c->d.B, c->l.es);
  return factors_into(c, W, X, aux, u, v, c->d.model == SFB_SC ? global_codes(aux, c->d.B) : CsrView());
}

int sfb_pack(sfb_ctx* c, const void* U, const void* V, const sfb_aux* aux, void* sf_buf, uint32_t clock) {
  if (c == nullptr || U == nullptr || sf_buf == nullptr) return SFB_ERR_ARG;
  if (!aligned(U, 16) || !aligned(sf_buf, 128)) return SFB_ERR_ARG;
  const sfb_desc& d = c->d;
  const uint32_t* rowptr = nullptr;
  if (d.v_sparse) {
    if (aux == nullptr || aux->rowptr == nullptr || aux->idx == nullptr || aux->val == nullptr) return SFB_ERR_ARG;
    rowptr = aux->rowptr;
  } else if (V == nullptr || !aligned(V, 16)) {
    return SFB_ERR_ARG;
  }
  ACC(launch_copy_rows(c->stream, caller_rows(U, c->l.ldu, d.B, c->l.es), stream_u(c, sf_buf), c->K, d.J));
  if (d.v_sparse)
    ACC(launch_pack_csr(c->stream, sf_buf, d, c->l, aux->rowptr, aux->idx, reinterpret_cast<const float*>(aux->val),
                        c->dev_status));
  else
    ACC(launch_copy_rows(c->stream, caller_rows(V, c->l.ldv, d.B, c->l.es), stream_v(c, sf_buf), c->K, d.D));
  ACC(launch_write_header(c->stream, sf_buf, d, c->l, clock, rowptr));
  if (d.compact) ACC(launch_compact(c->stream, sf_buf, d, c->l, c->compact_ws));
  return SFB_OK;
}

// csc_built: the atom-major re-sort of this buffer's codes for these K samples is already in the workspace
// active_rows: c->dml_active describes the u rows of this buffer (set by the factor stage of the same step)
static int apply_from(sfb_ctx* c, void* W, const void* sf_buf, float eta, int K, bool check, bool csc_built = false,
                      bool active_rows = false) {
  const sfb_desc& d = c->d;
  if (check) ACC(launch_check_header(c->stream, sf_buf, d, c->l, c->dev_status));
  if (d.v_sparse && d.path == SFB_PATH_F32 && c->csc_ws != nullptr) {
    if (!csc_built)
      ACC(launch_sc_csc_build(c->stream, stream_codes(c, sf_buf), K, d.D, (long long)d.nnz_capacity, c->csc_ws,
                              c->dev_status));
    ACC(launch_sc_csc_apply(c->stream, reinterpret_cast<float*>(W), stream_u(c, sf_buf), K, d.J, d.D, eta,
                            (long long)d.nnz_capacity, c->csc_ws, c->dev_status));
  } else if (d.v_sparse && d.path == SFB_PATH_F32) {
    ACC(launch_sc_apply(c->stream, reinterpret_cast<float*>(W), stream_codes(c, sf_buf), stream_u(c, sf_buf), K, d.J,
                        d.D, eta, c->dev_status, c->dev_status));
  } else if (d.v_sparse) {
    // dense alternative: rebuild the dense code rows from the buffer's CSR streams unless this step just made them
    if (check)
      ACC(launch_densify_codes(c->stream, stream_codes(c, sf_buf), dense_codes(c), K, d.D, c->dev_status,
                               d.path == SFB_PATH_TF32));
    ACC(umma_apply(c->umma, c->stream, W, has_shadow(c) ? c->w_shadow : nullptr, stream_u(c, sf_buf), dense_codes(c), eta,
                   K, c->dev_status));
    if (has_shadow(c)) c->shadow_of = W;   // the apply epilogue rewrote the shadow from the new W
  } else if (d.path == SFB_PATH_F32) {
    const int* idx = nullptr;
    const int* n_idx = nullptr;
    if (d.compact) {   // compacted buffer: the kept pairs sit in the first n_sf slots of every worker (directory)
      ACC(launch_kept_rows(c->stream, sf_buf, d.B, K / d.B, c->kept_idx, c->kept_idx + c->K));
      idx = c->kept_idx;
      n_idx = c->kept_idx + c->K;
    } else if (active_rows && c->dml_active != nullptr) {   // ordered list of the contributing pairs among the first K
      ACC(launch_compact_active(c->stream, c->dml_active, K, c->dml_idx, c->dml_idx + c->K));
      idx = c->dml_idx;
      n_idx = c->dml_idx + c->K;
    }
    ACC(launch_apply_f32(c->stream, reinterpret_cast<float*>(W), stream_u(c, sf_buf), stream_v(c, sf_buf), K, d.J, d.D,
                         eta, c->dev_status, idx, n_idx));
  } else {
    ACC(umma_apply(c->umma, c->stream, W, c->w_shadow, stream_u(c, sf_buf), stream_v(c, sf_buf), eta, K, c->dev_status,
                   d.compact ? reinterpret_cast<const char*>(sf_buf) + 128 : nullptr));
    // The apply epilogue rewrote the shadow from the new W.  (A compacted buffer without a single pair launches no
    // tile: W and a shadow that mirrored it stay as they were; a stale shadow stays stale.)
    if (has_shadow(c) && (!d.compact || c->shadow_of == W)) c->shadow_of = W;
    else c->shadow_of = nullptr;
  }
  return SFB_OK;
}

int sfb_factors_shard(sfb_ctx* c, const void* W, const void* X, const sfb_aux* aux, void* sf_buf, int32_t first_worker,
                      int32_t n_workers) {
  if (c == nullptr || W == nullptr || sf_buf == nullptr) return SFB_ERR_ARG;
  if (!aligned(W, 16) || !aligned(sf_buf, 128)) return SFB_ERR_ARG;
  const sfb_desc& d = c->d;
  if (first_worker < 0 || n_workers <= 0 || first_worker > d.P - n_workers) return SFB_ERR_ARG;
  int r = check_aux(c, aux);
  if (r != SFB_OK) return r;
  if (d.model != SFB_SC && (X == nullptr || !aligned(X, 16))) return SFB_ERR_ARG;
  // the shard's streams: every offset below is relative to the first of them
  char* shard = reinterpret_cast<char*>(sf_buf) + (long long)first_worker * c->l.stream_stride;
  CsrView codes;
  memset(&codes, 0, sizeof(codes));
  if (d.v_sparse) {
    sfb_desc ds = d;
    ds.P = n_workers;
    ACC(launch_pack_csr(c->stream, shard, ds, c->l, aux->rowptr, aux->idx, reinterpret_cast<const float*>(aux->val),
                        c->dev_status));
    codes = stream_codes(c, shard);
  }
  r = factors_into(c, W, X, aux, stream_u(c, shard), d.v_sparse ? RowMap() : stream_v(c, shard), codes, n_workers);
  if (r < 0) return r;
  // a process compacts the streams of its own workers before they are sent
  if (d.compact) ACC(launch_compact(c->stream, sf_buf, d, c->l, c->compact_ws, first_worker, n_workers));
  return SFB_OK;
}

int sfb_commit_header(sfb_ctx* c, void* sf_buf, uint32_t clock) {
  if (c == nullptr || sf_buf == nullptr || !aligned(sf_buf, 128)) return SFB_ERR_ARG;
  ACC(launch_write_header(c->stream, sf_buf, c->d, c->l, clock, nullptr));
  // compacted streams: the directory is local, its pair counts are rebuilt from what the exchange brought
  if (c->d.compact) ACC(launch_count_pairs(c->stream, sf_buf, c->d, c->l, c->compact_ws));
  return SFB_OK;
}

int sfb_apply(sfb_ctx* c, void* W, const void* sf_buf, float eta, int32_t K) {
  if (c == nullptr || W == nullptr || sf_buf == nullptr) return SFB_ERR_ARG;
  if (!aligned(W, 16) || !aligned(sf_buf, 128)) return SFB_ERR_ARG;
  if (K <= 0 || K > c->K || (K % c->d.B) != 0) return SFB_ERR_ARG;
  if (has_shadow(c) && c->shadow_of != W) c->shadow_of = nullptr;
  if (c->umma != nullptr) umma_drop_corr(c->umma);   // the buffer is the caller's: nothing prepared for it counts
  return apply_from(c, W, sf_buf, eta, K, true);
}

int sfb_step(sfb_ctx* c, void* W, const void* X, const sfb_aux* aux, void* sf_buf, float eta, int32_t K,
             uint32_t clock) {
  if (c == nullptr || W == nullptr || sf_buf == nullptr) return SFB_ERR_ARG;
  if (!aligned(W, 16) || !aligned(sf_buf, 128)) return SFB_ERR_ARG;
  if (K <= 0 || K > c->K || (K % c->d.B) != 0) return SFB_ERR_ARG;
  int r = check_aux(c, aux);
  if (r != SFB_OK) return r;
  const sfb_desc& d = c->d;
  if (d.model != SFB_SC && (X == nullptr || !aligned(X, 16))) return SFB_ERR_ARG;
  CsrView codes;
  memset(&codes, 0, sizeof(codes));
  const int slot = c->prof_n % 128;
  if (c->profiling) cudaEventRecord(c->prof_ev[slot][0], c->stream);
  // What does not depend on the factors goes to the auxiliary stream, beside the forward pass: the codes into
  // the buffer, header and directory, and the atom-major re-sort of the codes for the scatter apply.
  bool forked = false;
  if (c->aux_ok) {
    if (cudaEventRecord(c->aux_fork, c->stream) != cudaSuccess || cudaStreamWaitEvent(c->aux, c->aux_fork, 0) != cudaSuccess)
      return SFB_ERR_CUDA;
    forked = true;
  }
  cudaStream_t hs = forked ? c->aux : c->stream;
  bool csc_built = false;
  // From here on the auxiliary stream may hold work of this call: every exit joins it first (join_aux), so that the
  // context's stream never runs ahead of it and a stream capture in progress stays well formed.
  auto aux_side = [&]() -> int {
    if (d.v_sparse) {
      ACC(launch_pack_csr(hs, sf_buf, d, c->l, aux->rowptr, aux->idx, reinterpret_cast<const float*>(aux->val),
                          c->dev_status));
      // the forward reads the codes it just committed to the buffer, or, beside the packing, the caller's arrays
      // cut to the same per-worker capacity (so u always belongs to the codes that are on the wire and applied)
      codes = forked ? global_codes(aux, d.B, c->l.cap_p) : stream_codes(c, sf_buf);
    }
    ACC(launch_write_header(hs, sf_buf, d, c->l, clock, d.v_sparse ? aux->rowptr : nullptr));
    if (forked && d.v_sparse && d.path == SFB_PATH_F32 && c->csc_ws != nullptr) {
      ACC(launch_sc_csc_build(hs, stream_codes(c, sf_buf), K, d.D, (long long)d.nnz_capacity, c->csc_ws, c->dev_status));
      csc_built = true;
    }
    return SFB_OK;
  };
  auto join_aux = [&]() -> int {
    if (!forked) return SFB_OK;
    if (cudaEventRecord(c->aux_join, c->aux) != cudaSuccess || cudaStreamWaitEvent(c->stream, c->aux_join, 0) != cudaSuccess)
      return SFB_ERR_CUDA;
    return SFB_OK;
  };
  r = aux_side();
  if (r < 0) {
    join_aux();
    return r;
  }
  // the join event is recorded before the forward pass is enqueued, so the wait below covers exactly the side work
  if (forked && cudaEventRecord(c->aux_join, c->aux) != cudaSuccess) {
    join_aux();
    return SFB_ERR_CUDA;
  }
  r = factors_into(c, W, X, aux, stream_u(c, sf_buf), d.v_sparse ? RowMap() : stream_v(c, sf_buf), codes, 0,
                   d.path == SFB_PATH_TF32X3 && !d.compact && K == c->K);
  if (forked && cudaStreamWaitEvent(c->stream, c->aux_join, 0) != cudaSuccess) return SFB_ERR_CUDA;
  if (r < 0) return r;
  // pairs whose u came out as zero are dropped from the message before it is "sent" (and applied)
  if (d.compact) ACC(launch_compact(c->stream, sf_buf, d, c->l, c->compact_ws));
  if (c->profiling) cudaEventRecord(c->prof_ev[slot][1], c->stream);
  const bool listed = !d.compact && d.model == SFB_DML && d.path == SFB_PATH_F32 && c->dml_active != nullptr &&
                      (long long)((d.J + 127) / 128) * ((d.D + 127) / 128) >= 148;   // the large-tile apply takes the list
  r = apply_from(c, W, sf_buf, eta, K, false, csc_built, listed);
  c->last_step_K = K;
  c->last_step_listed = listed;
  if (c->profiling) {
    cudaEventRecord(c->prof_ev[slot][2], c->stream);
    c->prof_n++;
  }
  return r;
}

// Copies `bytes` from host memory into staging buffer `slot` of set `set` (grown on demand) on the copy stream.
static int stage_in(sfb_ctx* c, int set, int slot, const void* host, size_t bytes, const void** dev) {
  if (bytes > c->host_stage_bytes[set][slot]) {
    if (c->host_stage[set][slot]) {
      cudaStreamSynchronize(c->stream);   // the old buffer may still be in use by an earlier step
      cudaStreamSynchronize(c->copy_stream);
      cudaFree(c->host_stage[set][slot]);
      c->host_stage[set][slot] = nullptr;
      c->host_stage_bytes[set][slot] = 0;
    }
    if (cudaMalloc(&c->host_stage[set][slot], bytes) != cudaSuccess) {
      cudaGetLastError();
      return SFB_ERR_ALLOC;
    }
    c->host_stage_bytes[set][slot] = bytes;
  }
  if (cudaMemcpyAsync(c->host_stage[set][slot], host, bytes, cudaMemcpyHostToDevice, c->copy_stream) != cudaSuccess)
    return SFB_ERR_CUDA;
  *dev = c->host_stage[set][slot];
  return SFB_OK;
}

int sfb_step_host(sfb_ctx* c, void* W, const void* X_host, const sfb_aux* aux_host, void* sf_buf, float eta, int32_t K,
                  uint32_t clock, void* header_host) {
  if (c == nullptr || W == nullptr || sf_buf == nullptr || aux_host == nullptr) return SFB_ERR_ARG;
  const sfb_desc& d = c->d;
  const size_t es = (size_t)c->l.es, Kt = (size_t)c->K;
  sfb_aux dev_aux;
  memset(&dev_aux, 0, sizeof(dev_aux));
  const void* X_dev = nullptr;
  int r;
  if (!c->host_ready) {
    if (cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return SFB_ERR_CUDA;
    for (int k = 0; k < 2; ++k)
      if (cudaEventCreateWithFlags(&c->copied[k], cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&c->consumed[k], cudaEventDisableTiming) != cudaSuccess)
        return SFB_ERR_CUDA;
    c->host_ready = true;
  }
  const int set = (int)(c->host_steps & 1);
  // this set's buffers were last read by the step two calls ago
  if (c->host_steps >= 2 && cudaStreamWaitEvent(c->copy_stream, c->consumed[set], 0) != cudaSuccess) return SFB_ERR_CUDA;
  if (d.model != SFB_SC) {
    if (X_host == nullptr) return SFB_ERR_ARG;
    if ((r = stage_in(c, set, 0, X_host, Kt * d.D * es, &X_dev)) != SFB_OK) return r;
  }
  const void* p = nullptr;
  if (d.model == SFB_MLR) {
    if (aux_host->labels == nullptr) return SFB_ERR_ARG;
    if ((r = stage_in(c, set, 1, aux_host->labels, Kt * 4, &p)) != SFB_OK) return r;
    dev_aux.labels = static_cast<const int32_t*>(p);
    dev_aux.dual = aux_host->dual;          // SDCA state lives on the device
    dev_aux.sdca_step = aux_host->sdca_step;
  } else if (d.model == SFB_DML) {
    if (aux_host->Xb == nullptr || aux_host->similar == nullptr) return SFB_ERR_ARG;
    if ((r = stage_in(c, set, 1, aux_host->Xb, Kt * d.D * es, &p)) != SFB_OK) return r;
    dev_aux.Xb = p;
    if ((r = stage_in(c, set, 2, aux_host->similar, Kt, &p)) != SFB_OK) return r;
    dev_aux.similar = static_cast<const uint8_t*>(p);
  } else {
    if (!aux_host->rowptr || !aux_host->idx || !aux_host->val || !aux_host->Xdata) return SFB_ERR_ARG;
    const size_t nnz = aux_host->rowptr[Kt];   // host memory: readable here
    if (nnz > d.nnz_capacity) return SFB_ERR_SHAPE;
    if ((r = stage_in(c, set, 1, aux_host->rowptr, (Kt + 1) * 4, &p)) != SFB_OK) return r;
    dev_aux.rowptr = static_cast<const uint32_t*>(p);
    if ((r = stage_in(c, set, 2, aux_host->idx, (nnz > 0 ? nnz : 1) * 4, &p)) != SFB_OK) return r;
    dev_aux.idx = static_cast<const uint32_t*>(p);
    if ((r = stage_in(c, set, 3, aux_host->val, (nnz > 0 ? nnz : 1) * 4, &p)) != SFB_OK) return r;
    dev_aux.val = p;
    if ((r = stage_in(c, set, 4, aux_host->Xdata, Kt * d.J * 4, &p)) != SFB_OK) return r;
    dev_aux.Xdata = p;
  }
  if (cudaEventRecord(c->copied[set], c->copy_stream) != cudaSuccess) return SFB_ERR_CUDA;
  if (cudaStreamWaitEvent(c->stream, c->copied[set], 0) != cudaSuccess) return SFB_ERR_CUDA;
  if ((r = sfb_step(c, W, X_dev, &dev_aux, sf_buf, eta, K, clock)) != SFB_OK) return r;
  if (cudaEventRecord(c->consumed[set], c->stream) != cudaSuccess) return SFB_ERR_CUDA;
  ++c->host_steps;
  if (header_host != nullptr &&
      cudaMemcpyAsync(header_host, sf_buf, 128, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess)
    return SFB_ERR_CUDA;
  return SFB_OK;
}

}  // extern "C"
