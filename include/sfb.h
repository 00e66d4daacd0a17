/*
 * sfb.h -- C ABI of the sufficient-factor (SF) hot path on one NVIDIA B200 (sm_100a).
 *
 * The library computes, for matrix-parametrised models min_W (1/N) sum_i f_i(W a_i) + h(W)
 * (paper Section 2, problem (P), W in R^{J x D}), the two stages of Sufficient Factor
 * Broadcasting that touch W:
 *
 *   1. per-sample sufficient factors (u_i, v_i) with  grad_i = u_i v_i^T,
 *      u_i = d f_i / d (W a_i),  v_i = a_i                       (Section 2.1, "Proximal SGD");
 *   2. the rank-K update from the factors of all P workers,
 *      W <- W - eta * sum_{i<K} u_i v_i^T,  K = P*B               (Section 3, incl. "Mini-batch").
 *
 * Between the two sits the SF buffer: the message the P workers would broadcast, laid out as P
 * worker streams in one device buffer (Section 4.2: write_u / write_v / commit; Section 4.4:
 * input/output SF queues).  No network is involved; the P workers are simulated in one buffer.
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller and 128-byte aligned.  The
 *     library never frees or reallocates caller memory; it allocates only its own workspace, in
 *     sfb_create, and frees it in sfb_destroy.
 *   - All calls enqueue work on the CUDA stream given to sfb_create and return without
 *     synchronising, except sfb_status and sfb_destroy.
 *   - Return value: 0 (SFB_OK) or a negative SFB_ERR_* code found on the host before anything was
 *     launched (no partial effect).  Conditions only the device can see (label out of range, CSR
 *     index out of range or unsorted, SF-buffer header not matching the descriptor, CSR capacity
 *     exceeded) set bits of a sticky device status word and make the kernel that found them skip
 *     the affected writes; nothing traps.  Read the word with sfb_status.
 *   - A context is not thread-safe: calls on one context come from one host thread at a time.  Different
 *     contexts are independent (also on different devices of one process; a context belongs to the
 *     device that was current in sfb_create, which must be current again for every call on it).
 *   - sfb_compute_factors, sfb_pack, sfb_apply, sfb_step, sfb_factors_shard and sfb_commit_header only enqueue
 *     kernels (and event fork / join with a side stream of the context); after one ordinary call, which does
 *     the one-time kernel attribute set-up, a call may be recorded into a CUDA graph by capturing the context's
 *     stream and replayed (pointers and the clock are then the recorded ones, and so is the decision whether
 *     the context's cached copy of W, see sfb_invalidate, had to be rebuilt first: record a call that follows an
 *     ordinary call on the same W, and do not replay it after W was changed from outside).
 *   - "allocates only in sfb_create" has two stated exceptions, both on first use: the staging buffers
 *     of sfb_step_host and the workspace of sfb_loss.
 *   - W is J x D, row-major fp32, updated in place.  Samples are rows: X is [K][D].
 *   - Sample i belongs to worker p = i / B, slot i % B.
 *
 * Arithmetic paths (sfb_desc.path)
 *   SFB_PATH_F32   fp32 FMA on CUDA cores; X, U, V fp32.
 *   SFB_PATH_TF32  tensor cores (tcgen05, kind::tf32), fp32 accumulate; X, U, V fp32 in memory.
 *   SFB_PATH_BF16  tensor cores (tcgen05, kind::f16 with bf16 inputs), fp32 accumulate; X, U, V
 *                  bf16 in memory; W stays an fp32 master and the context keeps a bf16 shadow of
 *                  it that the apply refreshes.
 *   SFB_PATH_TF32X3  tensor cores with error compensation, for fp32-grade results (the tolerance class of
 *                  SFB_PATH_F32): every fp32 operand x is the part the tensor core sees (its top 10 mantissa
 *                  bits, hi) plus an exact remainder lo, and a product is formed as a b ~ hi hi + lo b + a lo:
 *                  hi hi by a tf32 multiplication of the operands as they are, the two corrections by one bf16
 *                  multiplication of "correction operands" [lo(a) | a] and [b | lo(b)] that a pre-pass (and,
 *                  for W, the apply's write-back) keeps in the context's workspace; X, U, V fp32 in memory,
 *                  same wire format as SFB_PATH_TF32.  The context caches W's correction operand like the
 *                  bf16 shadow (sfb_invalidate).  The tensor core's fp32 accumulator rounds toward zero
 *                  once per instruction of 8 reduction steps, which costs about 1.6e-8 of a sum per
 *                  instruction: forward reductions are cut into ranges that are added in fp32 afterwards, and
 *                  updates of more than 1024 pairs are applied to W in several launches of whole worker streams.
 *
 * SF buffer wire format (little-endian; every offset a multiple of 128 bytes)
 *   header, 128 bytes:
 *      0 u32 magic 0x31424653 ("SFB1")   4 u16 version 1   6 u8 model   7 u8 value dtype (0 f32, 1 bf16)
 *      8 u32 flags (bit 0: v is sparse)  12 u32 P  16 u32 B  20 u32 J  24 u32 D
 *     28 u32 clock (iteration number)    32 u32 ldu  36 u32 ldv
 *     40 u64 stream_stride  48 u64 total_bytes  56 u64 streams_off  64 u32 cap_p   rest zero
 *   directory at 128: P entries of 32 bytes {u32 worker, u32 n_sf (= B), u32 clock, u32 nnz,
 *      u64 u_off, u64 v_off}, padded to 128 bytes.
 *   worker stream p at streams_off + p * stream_stride:
 *      U block: B rows of ldu values, row r = u of sample p*B + r, pad values zero, padded to 128 B;
 *      V block: dense: B rows of ldv values; sparse (CSR): u32 rowptr[B+1] (local, starts at 0),
 *               u32 idx[cap_p], value val[cap_p], each padded to 128 B, unused tail zero.
 *   ldu (ldv) is J (D) rounded up so that a row is a whole number of 16-byte units.
 *   cap_p = nnz_capacity / P.  bf16 values are fp32 rounded to nearest even.
 *
 * Compacted buffers (sfb_desc.compact = 1; Section 6.1: the sufficient factors are sparse and that is used)
 *   A pair whose u is all zeros (a dissimilar DML pair beyond the margin, a sample with a bad label) adds nothing
 *   to the update and is not sent.  Per worker the remaining pairs sit in the first n_sf slots of the U and V
 *   blocks, in their original order; the slots behind them are zero; the directory's n_sf is the worker's own
 *   count and flags bit 1 is set.  Offsets and strides are those of the full buffer: a sender transmits the
 *   first n_sf rows of each block (sfb_wire_bytes counts them), a receiver reads them in place.  sfb_pack and
 *   sfb_step compact, sfb_apply leaves out the reduction blocks that hold only empty slots; W' is the same
 *   sum (bit-identical on SFB_PATH_F32).  In the sharded step every process compacts the streams of its own
 *   workers (sfb_factors_shard) before the exchange and sfb_commit_header rebuilds the pair counts from the streams
 *   that arrived.  Not available with sparse v.
 */
#ifndef SFB_H_
#define SFB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sfb_ctx sfb_ctx; /* opaque: workspace, cached tensor maps, device status word */

enum { SFB_MLR = 0, SFB_DML = 1, SFB_SC = 2 };
enum { SFB_PATH_F32 = 0, SFB_PATH_TF32 = 1, SFB_PATH_BF16 = 2, SFB_PATH_TF32X3 = 3 };

enum {
  SFB_OK = 0,
  SFB_ERR_ARG = -1,         /* null pointer, misaligned pointer, K not a whole number of worker streams */
  SFB_ERR_SHAPE = -2,       /* non-positive or unsupported sizes */
  SFB_ERR_UNSUPPORTED = -3, /* model/path combination not provided, or not an sm_100 device */
  SFB_ERR_CUDA = -4,        /* a CUDA runtime or driver call failed */
  SFB_ERR_ALLOC = -5,       /* workspace allocation failed */
  SFB_ERR_SCRATCH = -6      /* problem larger than the fixed scratch of sfb_sc_factors_noalloc */
};

/* bits of the device status word */
enum {
  SFB_DEV_BAD_LABEL = 1,    /* MLR label outside [0, J): that sample's u is written as zeros */
  SFB_DEV_BAD_INDEX = 2,    /* CSR column >= D or not strictly ascending: that entry is skipped */
  SFB_DEV_BAD_HEADER = 4,   /* SF buffer header does not match the descriptor: apply leaves W untouched */
  SFB_DEV_CAPACITY = 8,     /* a worker's nonzeros exceed cap_p: that stream's codes are truncated */
  SFB_DEV_TIMEOUT = 16      /* a bounded device-side wait (about a second) ran out: the launch completed, its
                               output is not to be used; the context stays usable */
};

typedef struct sfb_desc {
  int32_t model;         /* SFB_MLR / SFB_DML / SFB_SC */
  int32_t path;          /* SFB_PATH_* */
  int32_t J, D;          /* W is J x D (SC: J = feature dimension, D = number of atoms) */
  int32_t P, B;          /* simulated workers, SF pairs per worker; K = P*B */
  int32_t v_sparse;      /* 1: v is CSR (required for SFB_SC), 0: dense */
  float margin;          /* DML hinge margin on the squared distance */
  uint64_t nnz_capacity; /* total CSR capacity (a multiple of 32*P) when v_sparse */
  int32_t compact;       /* 1: pairs whose u is all zeros are left out of the SF buffer (dense v only), see below */
} sfb_desc;

/* Per-model side inputs of the factor computation (device pointers; unused ones NULL). */
typedef struct sfb_aux {
  const int32_t* labels;  /* MLR: class of each sample, [K] */
  const void* Xb;         /* DML: second element of each pair, [K][D], same type as X (X is the first) */
  const uint8_t* similar; /* DML: 1 = similar pair, 0 = dissimilar, [K] */
  const uint32_t* rowptr; /* SC: CSR row pointers of the codes, [K+1], rowptr[0] = 0 */
  const uint32_t* idx;    /* SC: atom index of each nonzero, strictly ascending within a row */
  const void* val;        /* SC: value of each nonzero (fp32) */
  const void* Xdata;      /* SC: data vectors x_i, [K][J] fp32 */
  void* dual;             /* MLR, optional: SDCA dual variables of the K samples (see below), DEVICE memory also for
                             sfb_step_host, [K][J rounded up to 4] fp32, updated in place; NULL = SGD factors */
  float sdca_step;        /* MLR with dual: damping of the dual step, in (0, 1] */
} sfb_aux;

/* Creates a context for one (model, path, shape).  `cuda_stream` is a cudaStream_t (NULL = the
 * legacy default stream).  Allocates the workspace the chosen path needs.  (No paper counterpart
 * beyond the constructor sfb_app(J, D, staleness) of Section 4.2.) */
int sfb_create(const sfb_desc* desc, void* cuda_stream, sfb_ctx** out);

/* Synchronises the stream and frees the workspace. */
int sfb_destroy(sfb_ctx* ctx);

/* Bytes the caller must allocate for the SF buffer of `desc` (0 on a bad descriptor). */
size_t sfb_sf_buffer_bytes(const sfb_desc* desc);

/* Padded row lengths (in values) of U and V rows; caller-side U / V arrays use them too. */
int sfb_ld(const sfb_desc* desc, int32_t* ldu, int32_t* ldv);

/* Sufficient factors of K = P*B samples (Section 2.1; Figures 2 and 3):
 *   MLR  z = W x,           u = softmax(z) - onehot(label),              v = x
 *   DML  d = x - xb, z = W d, u = +z (similar) | -z*[|z|^2 < margin] (dissimilar), v = d
 *   SC   z = W a (a = CSR code), u = z - xdata,                          v = a (not copied here)
 * W [J][D] fp32; X [K][D] (fp32, or bf16 on SFB_PATH_BF16); U out [K][ldu]; V out [K][ldv]
 * (V may be NULL for SC and is ignored).  Pad columns of U and V are written as zeros.
 *
 * SDCA for L2-regularised MLR (Section 2.1, "Stochastic DCA": dual variables u_i, auxiliary matrix
 * Z = (1/N) sum_i u_i a_i^T, W = Z / lambda, and the update of Z is again an outer product (du_i, a_i)).  With
 * aux->dual set the factors are the dual steps of the K samples, all from the same W,
 *   du_i = sdca_step * (dual_i + softmax(W x_i) - onehot(y_i)),   dual_i <- dual_i - du_i,   v_i = x_i
 * (the paper leaves du_i to "minimising the dual over u_i", which has no closed form for this loss: this damped
 * step toward the coordinate's optimality condition dual_i = -grad f_i is this library's reading), and the caller
 * applies them with eta = 1 / (lambda N): W <- W - eta sum_i du_i x_i^T keeps W = (1 / (lambda N)) sum_i dual_i x_i^T.
 * A sample with a label outside [0, J) takes no step. */
int sfb_compute_factors(sfb_ctx* ctx, const void* W, const void* X, const sfb_aux* aux, void* U, void* V);

/* Lays K (u, v) pairs out as P worker streams with header and directory: what the workers would
 * broadcast after commit() (Section 4.2).  U [K][ldu], V [K][ldv] in the path's value type; for
 * sparse v pass V = NULL and the CSR arrays through `aux`.  Pure data movement. */
int sfb_pack(sfb_ctx* ctx, const void* U, const void* V, const sfb_aux* aux, void* sf_buf, uint32_t clock);

/* Rank-K update W <- W - eta * sum_{i<K} u_i v_i^T from the first K/B worker streams of the SF
 * buffer (Section 3: every worker applies the factors of all workers).  K must be a positive
 * multiple of B and at most P*B.  The sum order is fixed, so results are bit-reproducible. */
int sfb_apply(sfb_ctx* ctx, void* W, const void* sf_buf, float eta, int32_t K);

/* One iteration as Section 3 states it for a worker under BSP (Section 4.1): compute the SF pairs of the
 * minibatch against the current W, commit them (the broadcast: here, all P simulated workers' streams
 * written straight into the SF buffer, header and directory included, with the given clock), then apply
 * the pairs of all workers, W <- W - eta * sum_i u_i v_i^T, over the first K slots.  K as in sfb_apply.
 * SFB_SC: if a worker's nonzeros exceed cap_p (SFB_DEV_CAPACITY), u is computed from the truncated codes,
 * the ones that are on the wire and that the apply uses. */
int sfb_step(sfb_ctx* ctx, void* W, const void* X, const sfb_aux* aux, void* sf_buf, float eta, int32_t K,
             uint32_t clock);

/* sfb_step for callers whose minibatch lives in HOST memory: X_host and the arrays inside aux_host
 * are host pointers (pinned memory keeps the copies asynchronous) with the shapes sfb_step
 * documents; they are copied to context-owned device staging buffers (two sets, allocated on
 * first use, grown on demand) on a side stream, so the copy for one call overlaps the kernels of
 * the previous call; the step then runs on the context's stream, and the 128-byte header the step
 * committed to the SF buffer is copied back into header_host (may be NULL).  W and sf_buf stay
 * device pointers.  Returns without synchronising; header_host is valid after the stream has
 * been synchronised (sfb_status does). */
int sfb_step_host(sfb_ctx* ctx, void* W, const void* X_host, const sfb_aux* aux_host, void* sf_buf, float eta,
                  int32_t K, uint32_t clock, void* header_host);

/* The step as P real workers take it (Section 3, "Sufficient factor broadcasting": every worker computes
 * the SF pairs of its own data shard against its full local copy of W, broadcasts them to all other
 * workers, and applies every worker's pairs to its copy; BSP, Section 4: all workers apply the same set of
 * pairs at every clock).  A process that owns workers [first_worker, first_worker + n_workers) of the P
 * in the descriptor calls, per clock,
 *   1. sfb_factors_shard: the pairs of ITS n_workers * B samples, written straight into those workers'
 *      streams of the P-worker SF buffer (X, aux: the shard's minibatch only, laid out as for
 *      sfb_compute_factors with P = n_workers; SFB_SC row pointers start at 0).  Other streams untouched.
 *   2. the exchange (the caller's: the worker streams are contiguous and equally long, so an all-gather
 *      over bytes [streams_off, streams_off + P * stream_stride) of the buffer, each process contributing
 *      the streams it owns, in place, is the whole broadcast; header bytes 40..47 and 56..63 hold
 *      stream_stride and streams_off, see sfb_sf_buffer_layout).
 *   3. sfb_commit_header (header and directory, identical on every process; the SFB_SC directory takes each
 *      worker's nonzero count from the stream it received) and sfb_apply with K = P * B.
 * With one process owning all P workers the three calls leave exactly the W and SF buffer of sfb_step.
 * The factors of a worker do not depend on which other workers share its process, except through the
 * tile geometry the library picks for the shard's size (a split reduction, the width of the partial
 * softmax tiles): bit-identical in most configurations, always far inside the path's tolerance.
 * Returns SFB_ERR_ARG for a worker range outside [0, P).  Nothing is exchanged by the library. */
int sfb_factors_shard(sfb_ctx* ctx, const void* W, const void* X, const sfb_aux* aux, void* sf_buf,
                      int32_t first_worker, int32_t n_workers);
int sfb_commit_header(sfb_ctx* ctx, void* sf_buf, uint32_t clock);

/* Byte range of the worker streams inside the SF buffer of a descriptor: streams_off = offset of worker
 * 0's stream, stream_stride = bytes per worker stream (both multiples of 128).  Host-only arithmetic. */
int sfb_sf_buffer_layout(const sfb_desc* desc, uint64_t* streams_off, uint64_t* stream_stride);

/* Proximal operator applied after the update (Section 2.1: prox_{eta h}; Section 3: "finally each
 * worker applies the proximal operator").  SFB_SC: h is the indicator of ||W_k||_2 <= 1 for every
 * column (atom) k, so each column whose norm exceeds 1 is divided by its norm and the others are
 * left bit-identical (Figure 3, function prox).  SFB_MLR / SFB_DML: h = 0, nothing to do (returns
 * SFB_OK without launching).  W [J][D] fp32 in place. */
int sfb_prox(sfb_ctx* ctx, void* W);

/* Minibatch objective at W, the function whose gradient the sufficient factors of this minibatch carry
 * (Section 3, problem (P): the sum over the minibatch of f_i(W a_i); the update of Section 3 is a gradient
 * step on it).  SFB_MLR: sum_i logsumexp(W x_i) - (W x_i)[y_i].  SFB_DML: sum_i 1/2 |L d_i|^2 for a similar
 * pair, 1/2 max(0, margin - |L d_i|^2) for a dissimilar one.  SFB_SC: sum_i 1/2 |W a_i - x_i|^2.
 * Arguments as sfb_compute_factors; loss: DEVICE pointer to one double (8-byte aligned), written on the
 * context's stream.  The products are formed in the context's math path (SFB_DML always on the fp32
 * path), reduced per sample in fp32 and over the samples in fp64, in a fixed order (bit-reproducible).
 * A monitoring helper outside the step: W, the SF buffer and the step's state are untouched.  The first
 * call allocates K x J floats of workspace (SFB_ERR_ALLOC if that fails); later calls allocate nothing.
 * A label outside [0, J) contributes 0 and sets SFB_DEV_BAD_LABEL. */
int sfb_loss(sfb_ctx* ctx, const void* W, const void* X, const sfb_aux* aux, double* loss);

/* Number of (u, v) pairs the last sfb_step actually multiplied through.  SFB_DML on SFB_PATH_F32 leaves out the
 * pairs whose u is zero (dissimilar pairs beyond the margin; the update is bit-identical to the sum over all K
 * slots, Section 6 notes that such sparsity can be used), and so does every context with compact = 1 (the count
 * is then the number of pairs the compaction kept); every other model / path applies all K slots and reports K.  Synchronises the stream.  *n is 0 before the first step. */
int sfb_active_pairs(sfb_ctx* ctx, int32_t* n);

/* Bytes a broadcast of this committed buffer would carry (Section 5.1 counts them per pair of workers: every
 * worker sends its K pairs of J + D values to P - 1 peers): header, directory entries, and per worker its first
 * n_sf rows of U and of dense V (sparse v: its B rows of U, B + 1 row pointers and nnz (index, value) pairs);
 * padding is not counted.  Synchronises the stream (reads the directory back). */
int sfb_wire_bytes(sfb_ctx* ctx, const void* sf_buf, uint64_t* bytes);

/* Tells the context that W was changed by someone else, so what it caches of W (the bf16 shadow of
 * SFB_PATH_BF16, the correction operand of SFB_PATH_TF32X3) is stale. */
int sfb_invalidate(sfb_ctx* ctx);

/* Synchronises the stream, returns the sticky device status word in *device_status and clears it. */
int sfb_status(sfb_ctx* ctx, int32_t* device_status);

/* Measurement aid: while enabled, sfb_step records CUDA events on the context's stream before the
 * factor stage, between the factor stage and the apply, and after the apply (at most the last 128
 * steps are kept).  sfb_stage_ms synchronises the stream and returns the summed durations of the
 * recorded steps and their count, then forgets them.  (No paper counterpart; Section 6.4 of the
 * paper breaks iteration time down by stage in the same spirit.) */
int sfb_profile(sfb_ctx* ctx, int enable);
int sfb_stage_ms(sfb_ctx* ctx, float* factors_ms, float* apply_ms, int32_t* steps);

/* Number of kernels this context has launched so far (for launch accounting). */
int64_t sfb_launch_count(const sfb_ctx* ctx);

const char* sfb_strerror(int code);

/* Halton-sequence broadcast (Section 4.3): the Q workers that worker p (zero-based) of P would
 * send its factor stream to, (p + floor(P f)) mod P for f = 1/2, 1/4, 3/4, 1/8, 3/8, ... in that
 * order, written to peers[0..Q).  Host-only; peers is a HOST array.  SFB_ERR_ARG on bad arguments. */
int sfb_halton_peers(int32_t P, int32_t Q, int32_t p, int32_t* peers);

/* Stale-synchronous rule (Section 4.1): 1 if worker p, having computed t_p batches and received
 * tau[q] batches from each of the P workers, may start its next batch (no q with
 * t_p - tau[q] > staleness), else 0.  staleness 0 = BSP, negative = unbounded (ASP).  Host-only;
 * tau is a HOST array.  Negative return = SFB_ERR_*. */
int sfb_ssp_may_proceed(int64_t t_p, const int64_t* tau, int32_t P, int64_t staleness);

/* Sparse-coding factors u_i = W a_i - x_i for callers that must not allocate device memory: code
 * that runs while its stream is being captured into a CUDA graph, latency-bound loops that cannot
 * afford the allocator's implicit synchronisation, and processes whose device memory was handed
 * out once, with a fixed budget, by an outer framework.  (The paper has no counterpart: this is a
 * packaging variant of sfb_compute_factors for SFB_SC, same kernels, same results.)
 *
 * It takes no context.  Its scratch, the atom-major copy of W, is a fixed 16 MiB device array
 * built into the library (every GPU that loads the library carries it until the process exits),
 * so D * roundup(J, 4) may be at most sfb_noalloc_max_scratch_floats() = 4 Mi values; larger
 * problems return SFB_ERR_SCRATCH and launch nothing.  The call itself never allocates or frees.
 *
 * W [J][D] fp32; rowptr [K+1], idx, val: CSR codes (fp32 values, strictly ascending indices);
 * Xdata [K][J] fp32; U out [K][ldu] fp32 with ldu >= J a multiple of 4 (every pad column up to ldu
 * is written as zero).  dev_status: optional device int that receives the SFB_DEV_* bits (cleared
 * by the call).  With NULL the bits go to a word inside the library that no call reads back: pass
 * a pointer if malformed codes must be noticed.  All pointers are device pointers of the caller.
 *
 * The first call on each device looks up the address of the built-in array (host threads that make
 * it at the same time are serialised); make that first call outside any stream capture.  All calls
 * share the array and it keeps the last call's contents: everything a call depends on is rewritten
 * by that call, but two calls whose kernels overlap on the GPU (different streams, or host threads
 * that enqueue at the same time on different streams) race on it, so keep them on one stream. */
int sfb_sc_factors_noalloc(const void* W, int32_t J, int32_t D, int32_t K, const uint32_t* rowptr,
                           const uint32_t* idx, const void* val, const void* Xdata, void* U, int32_t ldu,
                           int32_t* dev_status, void* cuda_stream);
int64_t sfb_noalloc_max_scratch_floats(void);

#ifdef __cplusplus
}
#endif
#endif /* SFB_H_ */
