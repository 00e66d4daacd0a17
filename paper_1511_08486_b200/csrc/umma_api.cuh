// Tensor-core (tcgen05 / TMEM / TMA) side of the SF hot path: interface used by the C-ABI host code.
#pragma once

#include "common.cuh"

namespace sfb {

struct UmmaPlan;   // tensor maps and launch geometry for one descriptor

// Builds the plan for a TF32 or BF16 descriptor.
int umma_plan_create(const sfb_desc& d, const Layout& l, UmmaPlan** out);
void umma_plan_destroy(UmmaPlan* p);

// z = W a on the tensor cores followed by the model epilogue; factors go through u / v row maps.
// for_apply (compensated path): umma_apply of exactly these u / v rows, all K pairs, follows before anything else
// changes them: the kernels that write the factors also write the apply's correction operands (one use).
// workers > 0: only that many workers' samples (X, aux, u, v start at the first of them).
int umma_forward(UmmaPlan* p, cudaStream_t s, const void* W, const __nv_bfloat16* w_shadow, const void* X,
                 const sfb_aux* aux, RowMap u, RowMap v, int* dev_status, int workers = 0, bool for_apply = false);

// Z rows (fp32) = A rows (the path's value type) times Wop^T on the tensor cores; no epilogue beyond the store.
// w_corr: on the compensated path, W's correction operand (launch_split_k of W's rows, B side); w_shadow plays
// that part in umma_forward.
int umma_forward_rows(UmmaPlan* p, cudaStream_t s, const void* Wop, RowMap a, RowMap z, int* dev_status,
                      float2* stats = nullptr, int* n_parts_out = nullptr, int* part_cols_out = nullptr,
                      int* k_splits_out = nullptr, int max_splits = 1, long long split_stride = 0, int workers = 0,
                      const void* w_corr = nullptr, bool a_corr_ready = false);

// Sparse coding: u rows = dense code rows `a` (fp32) times W^T minus the data rows Xdata [K][J].
// a_corr: what umma_codes_corr returned, if the kernel that made the rows `a` has written it.
int umma_forward_sc(UmmaPlan* p, cudaStream_t s, const void* W, RowMap a, RowMap u, const float* Xdata, int* dev_status,
                    int workers = 0, const void* w_corr = nullptr, bool for_apply = false, const CorrOut* a_corr = nullptr);
// Compensated path: where the kernel that makes the dense code rows may write their correction operands (the
// forward's; with for_apply also the apply's, for which the code rows are the v rows).  Empty on other paths.
CorrOut umma_codes_corr(UmmaPlan* p, bool for_apply);

// Forgets correction operands a factor stage left for "its" apply (a caller that applies a buffer of its own).
void umma_drop_corr(UmmaPlan* p);

// W <- W - eta * U^T V on the tensor cores with the write-back (and bf16 shadow refresh) fused.
// u_rows / v_rows: the factor rows (normally the U and V blocks of the SF buffer's worker streams).
// directory (optional): the SF buffer's directory (sf_buf + 128) of a compacted buffer, whose rows behind each
// worker's pair count are zeros: reduction blocks that hold only such rows are skipped.
int umma_apply(UmmaPlan* p, cudaStream_t s, void* W, __nv_bfloat16* w_shadow, RowMap u_rows, RowMap v_rows, float eta,
               int K, const int* dev_status, const void* directory = nullptr);

}  // namespace sfb
