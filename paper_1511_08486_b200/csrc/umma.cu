// Tensor-core contractions of the SF hot path on sm_100a: tcgen05.mma with accumulators in tensor
// memory (TMEM), operands brought to shared memory by TMA, one persistent CTA per SM.
//
//   forward:  Z[i][j] = sum_d A[i][d] * W[j][d]        (z_i = W a_i; Section 2, problem (P))
//             both operands are contiguous along the reduction index d ("K-major").
//   apply  :  W[j][d] -= eta * sum_i U[i][j] * V[i][d]   (W <- W - eta * sum_i u_i v_i^T; Section 3)
//             the factors are stored one u_i / v_i per row, so both operands are contiguous along
//             the output index ("MN-major"); tcgen05 reads them in that form directly from the SF
//             buffer's worker streams, no transposed copy is made.
//
// Warp roles (320 threads): warp 0 issues TMA loads into a shared-memory ring of 3 to 8 stages, warp 1 issues
// the MMAs (one thread) into one of two TMEM accumulators, warps 2-9 drain the other accumulator
// (tcgen05.ld) and run the epilogue, so the write-back of tile t overlaps the MMAs of tile t+1.
// The error-compensated kernels (SPLIT, fp32-grade results from tf32 MMAs) add warps 10-13, which split every
// operand stage into what the tensor core sees of it and the exact remainder.
// Every wait on an mbarrier is bounded; a wait that runs out sets SFB_DEV_TIMEOUT and the CTA leaves
// through the common exit (TMEM freed) instead of hanging.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "umma.cuh"
#include "umma_api.cuh"

namespace sfb {

// extra passes implemented in finish.cu
int launch_finish_mlr_fused(cudaStream_t s, RowMap u, const float2* stats, int n_parts, int part_cols,
                            const int32_t* labels, int K, int J, int* dev_status, float* dual, float sdca_step);

namespace {

constexpr int BM = 128;          // rows per CTA tile = TMEM lanes
constexpr int NUM_THREADS = 320;         // TMA warp, MMA warp, 8 epilogue warps
constexpr int EPI_STAGE_BYTES = 8 * 4096;  // one swizzled 32 x 32 fp32 block per epilogue warp
constexpr int RING_BYTES = 192 * 1024;   // shared memory given to the operand ring
constexpr int MAX_STAGES = 8;
constexpr int MAX_DIR_WORKERS = 256;      // workers whose pair counts the apply can take from the directory
constexpr uint32_t WAIT_LIMIT = 1u << 20;   // polls of a bounded wait: a failed poll suspends about 1.4 us, so about 1.4 s

struct GemmParams {
  int m_tiles, n_tiles, k_blocks;   // m_tiles counts tiles of 128*CG rows; k_blocks counts blocks of BK reduction steps
  int k_splits, k_per_split;        // forward only: the reduction is cut in k_splits ranges of k_per_split blocks, each
  long long split_stride;           // range writing its partial products to z + split * split_stride bytes
  int a_policy, b_policy;   // L2 eviction policy of the operand loads (0 normal, 1 evict first, 2 evict last)
  int m_fastest;            // tile order: 1 = consecutive tiles share the B operand slab, 0 = share the A slab
  int group;                // tiles of the fast dimension walked before the slow one advances (0 = all)
  int B, P;                 // rows per worker / workers, geometry of the operand maps
  int m_bb, m_wp, m_tpw;    // forward: 128 A rows come as a box of m_bb rows x m_wp workers; 128-row units per worker
  int k_bb, k_wp, k_bpw;    // apply: a reduction block is k_bb rows x k_wp workers; blocks per worker
  int Mvalid, Nvalid;       // apply: (J, D)
  float* W;                 // apply: fp32 master, row stride ldw
  // apply: bf16 copy of the new W (or nullptr); compensated kernels: W's correction operand for the next forward
  // pass, [row][atom of 32 columns][32 values | 32 remainders], w_atoms atoms per row
  __nv_bfloat16* shadow;
  int w_atoms;
  long long ldw;
  float eta;
  RowMap z;                 // forward: output rows (fp32 products, or exps in the factor's storage type)
  float2* stats;            // forward, EPI 1: (max, sum of exps) per (sample, half tile), [K][n_parts]
  int n_parts;
  // apply: directory of the SF buffer (32-byte entries, word 1 = the worker's pair count) when the rows behind a
  // worker's count are known to be zero and whole reduction blocks of them can be left out; nullptr = all B rows
  const uint32_t* dir;
  const int* status_ro;
  int* status;
  int lose_signal;          // test hook: the first pair / CTA drops its first "stage free" signal (see UmmaPlan)
};

struct SharedCtl {
  uint64_t full[MAX_STAGES], empty[MAX_STAGES], tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  volatile int abort;
  int k_total;                 // apply: reduction blocks per tile (sum of nb[] when a directory is given)
  uint16_t nb[MAX_DIR_WORKERS];   // apply with a directory: reduction blocks of each worker
};

__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, SharedCtl* ctl, int* status) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && ctl->abort) return false;
  }
  ctl->abort = 1;
  if (status != nullptr) atomicOr(status, SFB_DEV_TIMEOUT);
  return false;
}

// Tile order.  m_fastest = 0: consecutive tiles walk `group` column tiles, then the next row tile,
// and only after all row tiles the next group of columns; so one wave of CTAs touches few B slabs
// (they stay in L2 across waves) while the A slabs stream.  m_fastest = 1: the same with rows and
// columns exchanged.  group = 0 means one group spanning the whole dimension.
__device__ __forceinline__ void tile_coords(const GemmParams& p, int tile, int& mt, int& nt) {
  if (!p.m_fastest) {
    const int g = p.group > 0 ? p.group : p.n_tiles;
    const int per = p.m_tiles * g;
    const int sc = tile / per, r = tile - sc * per;
    const int ge = min(g, p.n_tiles - sc * g);
    mt = r / ge;
    nt = sc * g + (r - mt * ge);
  } else {
    const int g = p.group > 0 ? p.group : p.m_tiles;
    const int per = p.n_tiles * g;
    const int sc = tile / per, r = tile - sc * per;
    const int ge = min(g, p.m_tiles - sc * g);
    nt = r / ge;
    mt = sc * g + (r - nt * ge);
  }
}

// Template parameters of the GEMM kernel:
//   ES     bytes per operand value (2 = bf16, 4 = tf32); CH = 128 / ES values make one 128-byte chunk.
//   APPLY  MN-major operands (factor rows) and the W write-back epilogue; otherwise K-major operands
//          (sample rows / W rows) and a plain fp32 store of Z.
//   BN     tile columns.
//   CG     CTAs per MMA.  With CG = 2 the kernel runs as clusters of two CTAs on a 256 x BN tile: each
//          CTA loads its own 128 rows of A and its own half of B's columns, the even CTA issues
//          tcgen05.mma.cta_group::2 (M = 256) for the pair, each CTA drains its own 128 accumulator
//          rows.  TMA bytes of both CTAs are credited to the even CTA's "full" barrier; "stage free"
//          and "accumulator ready" are committed (tcgen05.commit) once to the even CTA's barrier and
//          once to the odd CTA's; both epilogues arrive on the even CTA's "accumulator drained" barrier.
//   KA     128-byte atoms of the reduction index per pipeline stage (BK = KA * CH reduction steps).
//   EPI    forward epilogue: 0 = store the products z; 1 = multiclass-logistic epilogue: store
//          exp(z - m) with m the row maximum over this warp's half tile, in the factor's storage
//          type, plus (m, sum of exps) per (sample, half tile) for the finishing pass that
//          rescales to the softmax and subtracts the one-hot label (Section 2.1: u = softmax - onehot).
//   FOLD   operands come through 4-D tensor maps whose extra dimension walks the 128-byte chunks, so
//          one TMA instruction fills a whole operand stage (needs J, D multiples of CH); otherwise
//          one 3-D TMA per chunk, with zero fill on every ragged edge.
//   SPLIT  error-compensated tf32 (ES = 4): the tensor core drops the low 13 mantissa bits of an fp32 operand, so
//          x = hi + lo with hi = what the tensor core sees of x and lo = x - hi (exact in fp32).  Besides its
//          fp32 operand tiles a stage then holds the bf16 correction tiles [lo(a) | a] and [b | lo(b)] (a
//          pre-pass writes them to global memory with the tiling of the fp32 operands, tensor maps tmAc / tmBc;
//          64 bf16 reduction steps per 128-byte atom of 32 fp32 ones), and every atom issues four tf32
//          instructions a * b into the main accumulator and four bf16 instructions lo(a) b + a lo(b) into a
//          second one (lo * lo, about 2^-22 of the product, is dropped; bf16 carries the corrections, themselves
//          2^-10 of the product, to 2^-18).  The accumulators are added in the epilogue.
//          Two accumulators because the tensor core's fp32 accumulation rounds toward zero once per
//          instruction (measured: a sum of n instructions comes out short by about n * 2^-26): the small
//          corrections must not cost the large sum more roundings.
template <int ES, bool APPLY, int BN, int CG, int KA, bool FOLD, int EPI, bool SPLIT>
__global__ void __launch_bounds__(NUM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmAc,
                 const __grid_constant__ CUtensorMap tmBc, const GemmParams p) {
  constexpr int CH = 128 / ES;                 // values per 128-byte chunk
  constexpr int BK = CH * KA;                  // reduction steps per pipeline stage
  constexpr int UMMA_K = 32 / ES;              // reduction steps per instruction (16 bf16 / 8 tf32)
  constexpr int BNC = BN / CG;                 // B columns this CTA loads
  constexpr int A_STAGE_BYTES = BM * 128 * KA;
  constexpr int B_STAGE_BYTES = BNC * 128 * KA;
  constexpr int RAW_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;     // what TMA brings per stage
  constexpr int STAGE_BYTES = RAW_BYTES * (SPLIT ? 2 : 1);     // SPLIT: the correction tiles follow, same sizes
  constexpr int NACC = SPLIT ? 2 : 1;                          // accumulators per tile (main, corrections)
  constexpr int ACC_COLS = BN * NACC;
  constexpr int NBUF = (2 * ACC_COLS <= 512) ? 2 : 1;          // accumulator sets in the 512 columns of tensor memory
  static_assert(!SPLIT || (ES == 4 && EPI == 0), "error compensation is for fp32 operands and plain stores");
  // whose "full" barrier a CTA's loads are credited to: its own, or the even CTA's (pairs: one barrier for the
  // MMA issuer)
  constexpr bool OWN = (CG == 1);
  constexpr int STAGES = (RING_BYTES / STAGE_BYTES) < MAX_STAGES ? (RING_BYTES / STAGE_BYTES) : MAX_STAGES;
  constexpr uint32_t IDESC = ptx::instr_desc(ES == 2 ? 1u : 2u, APPLY ? 1u : 0u, APPLY ? 1u : 0u, BM * CG, BN);
  constexpr uint32_t IDESC_C = ptx::instr_desc(1u, APPLY ? 1u : 0u, APPLY ? 1u : 0u, BM * CG, BN);   // SPLIT: bf16 corrections
  static_assert(!SPLIT || KA == 1, "the correction tiles hold one atom of the reduction");
  static_assert(STAGES >= 2, "ring too shallow");

  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* epi_stage = reinterpret_cast<float*>(tiles + STAGES * STAGE_BYTES);
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(tiles + STAGES * STAGE_BYTES + EPI_STAGE_BYTES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (p.status_ro != nullptr && (*p.status_ro & SFB_DEV_BAD_HEADER)) return;   // uniform over the grid

  const uint32_t rank = (CG == 2) ? ptx::cluster_ctarank() : 0u;   // 0 = the CTA that issues the MMAs
  const int cluster_id = blockIdx.x / CG, num_clusters = gridDim.x / CG;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&ctl->full[s], 1);
      ptx::mbar_init(&ctl->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&ctl->tmem_full[b], 1);
      ptx::mbar_init(&ctl->tmem_empty[b], 8 * CG);   // one arrival per epilogue warp of every CTA of the pair
    }
    ctl->abort = 0;
    if (APPLY) {
      int tot = p.k_blocks;
      if (p.dir != nullptr) {   // only with B >= BK and at most MAX_DIR_WORKERS workers (the host checks)
        tot = 0;
        for (int w = 0; w < p.P; ++w) {
          const int n = min((int)p.dir[w * 8 + 1], p.B);
          const int nbw = (n + BK - 1) / BK;
          ctl->nb[w] = (uint16_t)nbw;
          tot += nbw;
        }
      }
      ctl->k_total = tot;
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
    if (SPLIT) { ptx::prefetch_tmap(&tmAc); ptx::prefetch_tmap(&tmBc); }
  }
  if (warp == 1) {
    ptx::tmem_alloc<CG>(&ctl->tmem_base, NBUF * ACC_COLS);
    ptx::tmem_relinquish<CG>();
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (CG == 2) ptx::cluster_sync();   // the peer's barriers exist before anything is signalled remotely
  ptx::tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  // apply: every worker contributes its own number of reduction blocks; none at all = nothing to add to W
  const int k_blocks = APPLY ? ctl->k_total : p.k_blocks;
  const int k_per_split = APPLY ? k_blocks : p.k_per_split;
  const bool by_dir = APPLY && p.dir != nullptr;
  const int total_work = (APPLY && k_blocks == 0) ? 0 : p.m_tiles * p.n_tiles * p.k_splits;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (every CTA)
    int s = 0;
    uint32_t ph = 0;
    int issued = 0;
    bool ok = true;
    const uint64_t pol_a = ptx::l2_policy(p.a_policy), pol_b = ptx::l2_policy(p.b_policy);
    for (int work = cluster_id; work < total_work && ok; work += num_clusters) {
      const int tile = work / p.k_splits, split = work - tile * p.k_splits;
      const int kb_begin = split * k_per_split, kb_end = min(kb_begin + k_per_split, k_blocks);
      int mt, nt;
      tile_coords(p, tile, mt, nt);
      mt = mt * CG + (int)rank;                           // 128-row unit of this CTA
      const int ncol0 = nt * BN + (int)rank * BNC;       // first B column loaded here
      int slot0 = 0, mp0 = 0;          // forward: first slot / worker of this CTA's 128 sample rows
      if (!APPLY) {
        if (p.B >= BM) { mp0 = mt / p.m_tpw; slot0 = (mt % p.m_tpw) * BM; }
        else { mp0 = mt * p.m_wp; }
      }
      int row0 = 0, kp0 = 0;           // apply: first row / worker of the current reduction block
      if (by_dir)
        while (kp0 < p.P && ctl->nb[kp0] == 0) ++kp0;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        ok = wait_or_abort(&ctl->empty[s], ph ^ 1u, ctl, p.status);
        if (!ok) break;
        if (lane == 0) {
          uint8_t* a_dst = tiles + s * STAGE_BYTES;
          uint8_t* b_dst = a_dst + A_STAGE_BYTES;
          uint64_t* bar = &ctl->full[s];
          uint32_t full_addr = ptx::smem_u32(bar);
          if (CG == 2) full_addr = ptx::map_to_cta(full_addr, 0);
          if (OWN) ptx::mbar_expect_tx(bar, STAGE_BYTES);
          else if (rank == 0) ptx::mbar_expect_tx(bar, CG * STAGE_BYTES);
          if (!APPLY) {
            if (FOLD) {   // dims (value-in-atom, row, worker, atom): one box = KA atoms of 128 rows
              if (OWN) {
                ptx::tma_load_4d_hint(a_dst, &tmA, bar, 0, slot0, mp0, kb * KA, pol_a);
                ptx::tma_load_4d_hint(b_dst, &tmB, bar, 0, ncol0, 0, kb * KA, pol_b);
              } else {
                ptx::tma_load_4d_hint_pair(a_dst, &tmA, full_addr, 0, slot0, mp0, kb * KA, pol_a);
                ptx::tma_load_4d_hint_pair(b_dst, &tmB, full_addr, 0, ncol0, 0, kb * KA, pol_b);
              }
            } else {
#pragma unroll
              for (int a = 0; a < KA; ++a) {
                const int k0 = (kb * KA + a) * CH;
                if (OWN) {
                  ptx::tma_load_3d_hint(a_dst + a * (BM * 128), &tmA, bar, k0, slot0, mp0, pol_a);
                  ptx::tma_load_3d_hint(b_dst + a * (BNC * 128), &tmB, bar, k0, ncol0, 0, pol_b);
                } else {
                  ptx::tma_load_3d_hint_pair(a_dst + a * (BM * 128), &tmA, full_addr, k0, slot0, mp0, pol_a);
                  ptx::tma_load_3d_hint_pair(b_dst + a * (BNC * 128), &tmB, full_addr, k0, ncol0, 0, pol_b);
                }
              }
            }
          } else {
            if (FOLD) {   // dims (value-in-chunk, row, worker, chunk): one box = all chunks x BK rows
              if (OWN) {
                ptx::tma_load_4d_hint(a_dst, &tmA, bar, 0, row0, kp0, (mt * BM) / CH, pol_a);
                ptx::tma_load_4d_hint(b_dst, &tmB, bar, 0, row0, kp0, ncol0 / CH, pol_b);
              } else {
                ptx::tma_load_4d_hint_pair(a_dst, &tmA, full_addr, 0, row0, kp0, (mt * BM) / CH, pol_a);
                ptx::tma_load_4d_hint_pair(b_dst, &tmB, full_addr, 0, row0, kp0, ncol0 / CH, pol_b);
              }
            } else {
#pragma unroll
              for (int c = 0; c < BM / CH; ++c) {
                if (OWN) ptx::tma_load_3d_hint(a_dst + c * (BK * 128), &tmA, bar, mt * BM + c * CH, row0, kp0, pol_a);
                else ptx::tma_load_3d_hint_pair(a_dst + c * (BK * 128), &tmA, full_addr, mt * BM + c * CH, row0, kp0, pol_a);
              }
#pragma unroll
              for (int c = 0; c < BNC / CH; ++c) {
                if (OWN) ptx::tma_load_3d_hint(b_dst + c * (BK * 128), &tmB, bar, ncol0 + c * CH, row0, kp0, pol_b);
                else ptx::tma_load_3d_hint_pair(b_dst + c * (BK * 128), &tmB, full_addr, ncol0 + c * CH, row0, kp0, pol_b);
              }
            }
          }
        }
        if (SPLIT && lane == 0) {
          // correction tiles: same coordinates as the fp32 ones, in units of their own tiling
          uint8_t* ac_dst = tiles + s * STAGE_BYTES + RAW_BYTES;
          uint8_t* bc_dst = ac_dst + A_STAGE_BYTES;
          uint64_t* bar = &ctl->full[s];
          uint32_t full_addr = ptx::smem_u32(bar);
          if (CG == 2) full_addr = ptx::map_to_cta(full_addr, 0);
          if (!APPLY) {   // dims (value-in-atom, row, worker, atom)
            if (OWN) {
              ptx::tma_load_4d_hint(ac_dst, &tmAc, bar, 0, slot0, mp0, kb, pol_a);
              ptx::tma_load_4d_hint(bc_dst, &tmBc, bar, 0, ncol0, 0, kb, pol_b);
            } else {
              ptx::tma_load_4d_hint_pair(ac_dst, &tmAc, full_addr, 0, slot0, mp0, kb, pol_a);
              ptx::tma_load_4d_hint_pair(bc_dst, &tmBc, full_addr, 0, ncol0, 0, kb, pol_b);
            }
          } else {        // dims (value-in-chunk of 64, line, chunk): 64 lines per reduction block
            const int blk = (p.B >= BK) ? kp0 * p.k_bpw + row0 / BK : kp0 / p.k_wp;
            if (OWN) {
              ptx::tma_load_3d_hint(ac_dst, &tmAc, bar, 0, blk * 64, (mt * BM) / 64, pol_a);
              ptx::tma_load_3d_hint(bc_dst, &tmBc, bar, 0, blk * 64, ncol0 / 64, pol_b);
            } else {
              ptx::tma_load_3d_hint_pair(ac_dst, &tmAc, full_addr, 0, blk * 64, (mt * BM) / 64, pol_a);
              ptx::tma_load_3d_hint_pair(bc_dst, &tmBc, full_addr, 0, blk * 64, ncol0 / 64, pol_b);
            }
          }
        }
        if (APPLY) {   // next reduction block: next BK rows of this worker, or the next group of workers
          if (p.B >= BK) {
            row0 += BK;
            if (row0 >= (by_dir ? (int)ctl->nb[kp0] * BK : p.B)) {
              row0 = 0;
              ++kp0;
              if (by_dir)
                while (kp0 < p.P && ctl->nb[kp0] == 0) ++kp0;
            }
          } else {
            kp0 += p.k_wp;
          }
        }
        __syncwarp();
        ++issued;
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
    }
    if ((!ok || ctl->abort) && (rank == 0 || OWN)) {
      // let copies already in flight land before the CTA goes away (bounded)
      int n = issued < STAGES ? issued : STAGES;
      for (int q = 0; q < n; ++q) {
        int sq = s - 1 - q;
        uint32_t pq = ph;
        if (sq < 0) { sq += STAGES; pq ^= 1u; }
        ptx::mbar_wait(&ctl->full[sq], pq, 1u << 16);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (even CTA only)
    int s = 0;
    uint32_t ph = 0;
    int it = 0;
    bool ok = (rank == 0);
    for (int work = cluster_id; work < total_work && ok; work += num_clusters, ++it) {
      const int split = work % p.k_splits;
      const int kb_begin = split * k_per_split, kb_end = min(kb_begin + k_per_split, k_blocks);
      const int buf = it % NBUF;
      const uint32_t acc_ph = (uint32_t)(it / NBUF) & 1u;
      ok = wait_or_abort(&ctl->tmem_empty[buf], acc_ph ^ 1u, ctl, p.status);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t d_tmem = tmem_base + buf * ACC_COLS;
      const uint32_t d_lo = d_tmem + BN;              // SPLIT: accumulator of the correction products
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        ok = wait_or_abort(&ctl->full[s], ph, ctl, p.status);
        if (!ok) break;
        ptx::tc_fence_after();
        if (lane == 0) {
          const uint32_t a_addr = ptx::smem_u32(tiles + s * STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_STAGE_BYTES;
          if (!APPLY) {
            // K-major: a stage is KA atoms, each [rows][128 B] with 8-row groups 1024 B apart; inside an
            // atom the instruction's 32 bytes of reduction index advance the start address.
#pragma unroll
            for (int a = 0; a < KA; ++a) {
              const uint64_t a_desc = ptx::smem_desc(a_addr + a * (BM * 128), 16, 1024, 2);
              const uint64_t b_desc = ptx::smem_desc(b_addr + a * (BNC * 128), 16, 1024, 2);
#pragma unroll
              for (int k = 0; k < CH / UMMA_K; ++k) {
                const uint32_t acc = (kb > kb_begin || a > 0 || k > 0) ? 1u : 0u;
                if (ES == 2) ptx::mma_f16<CG>(d_tmem, a_desc + k * 2, b_desc + k * 2, IDESC, acc);
                else ptx::mma_tf32<CG>(d_tmem, a_desc + k * 2, b_desc + k * 2, IDESC, acc);
              }
              if (SPLIT) {
                // corrections: the bf16 tiles RAW_BYTES behind the fp32 ones, [lo(a) | a] times [b | lo(b)] over 64
                // reduction steps = lo(a) b + a lo(b) of the atom's 32; four instructions of 16
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  ptx::mma_f16<CG>(d_lo, a_desc + (RAW_BYTES >> 4) + k * 2, b_desc + (RAW_BYTES >> 4) + k * 2, IDESC_C,
                                   (kb > kb_begin || k > 0) ? 1u : 0u);
              }
            }
          } else {
            // MN-major: a stage is chunks of [BK reduction steps][128 B], BK*128 B apart; groups of 8
            // steps are 1024 B apart (32-bit values: 32-byte-atom swizzle, groups of 4 steps, 512 B).
            constexpr bool MN32 = ES == 4;
            const uint64_t a_desc = ptx::smem_desc(a_addr, BK * 128, MN32 ? 512 : 1024, MN32 ? 1 : 2);
            const uint64_t b_desc = ptx::smem_desc(b_addr, BK * 128, MN32 ? 512 : 1024, MN32 ? 1 : 2);
            constexpr uint32_t STEP = (UMMA_K * 128) >> 4;
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              const uint32_t acc = (kb > kb_begin || k > 0) ? 1u : 0u;
              if (ES == 2) ptx::mma_f16<CG>(d_tmem, a_desc + k * STEP, b_desc + k * STEP, IDESC, acc);
              else ptx::mma_tf32<CG>(d_tmem, a_desc + k * STEP, b_desc + k * STEP, IDESC, acc);
            }
            if (SPLIT) {
              // corrections: bf16 tiles of 64 reduction lines ([lo(a) ; a] and [b ; lo(b)]) in 128-byte chunks of 64
              // values, 8192 B apart, 128-byte swizzle; sixteen lines per instruction
              const uint64_t ac_desc = ptx::smem_desc(a_addr + RAW_BYTES, 64 * 128, 1024, 2);
              const uint64_t bc_desc = ptx::smem_desc(b_addr + RAW_BYTES, 64 * 128, 1024, 2);
#pragma unroll
              for (int k = 0; k < 4; ++k)
                ptx::mma_f16<CG>(d_lo, ac_desc + k * 128, bc_desc + k * 128, IDESC_C, (kb > kb_begin || k > 0) ? 1u : 0u);
            }
          }
          // (test hook: one lost signal, so that the producer's bounded wait runs out and the abort path is taken)
          const bool lost = p.lose_signal != 0 && cluster_id == 0 && it == 0 && kb == kb_begin;
          if (!lost) {
            ptx::mma_commit<CG>(&ctl->empty[s]);                   // stage reusable once these MMAs have read it
            if (CG == 2) ptx::mma_commit_addr<CG>(ptx::map_to_cta(ptx::smem_u32(&ctl->empty[s]), 1));
          }
          if (kb == kb_end - 1) {                                  // accumulator complete, in both CTAs
            ptx::mma_commit<CG>(&ctl->tmem_full[buf]);
            if (CG == 2) ptx::mma_commit_addr<CG>(ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_full[buf]), 1));
          }
        }
        __syncwarp();
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9, every CTA)
    // A warp may only read the TMEM lanes of its quarter (warp index mod 4).  Two warps share each
    // quarter and split the tile's columns in halves.  Per 32 x 32 block: accumulators come out of
    // TMEM one row per thread, go through an XOR-swizzled 4 KB shared-memory block, and are read back
    // four rows x 128 bytes per warp instruction, so that every global access is a full 128-byte line.
    const int e = warp - 2;
    const int quarter = warp & 3;
    const int half = e >> 2;
    float* stage = epi_stage + e * 1024;
    const int lrow = lane >> 3, lq = lane & 7;    // transposed assignment: row-in-group, 16-byte column
    int it = 0;
    bool ok = true;
    for (int work = cluster_id; work < total_work && ok; work += num_clusters, ++it) {
      const int tile = work / p.k_splits, split = work - tile * p.k_splits;
      int mt, nt;
      tile_coords(p, tile, mt, nt);
      mt = mt * CG + (int)rank;
      const int buf = it % NBUF;
      const uint32_t acc_ph = (uint32_t)(it / NBUF) & 1u;
      // destination rows of the 8 row groups this lane touches (row = quarter*32 + 4*g + lrow)
      float* rowp[8];
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        const int r = quarter * 32 + 4 * g + lrow;
        rowp[g] = nullptr;
        if (APPLY) {
          const int j = mt * BM + r;
          if (j < p.Mvalid) rowp[g] = p.W + (long long)j * p.ldw;
        } else {
          int wp_, slot;
          if (p.B >= BM) { wp_ = mt / p.m_tpw; slot = (mt % p.m_tpw) * BM + r; }
          else { wp_ = mt * p.m_wp + r / p.m_bb; slot = r % p.m_bb; }
          if (wp_ < p.P && slot < p.B)
            rowp[g] = reinterpret_cast<float*>(p.z.row(wp_ * p.B + slot) + split * p.split_stride);
        }
      }
      const int ncols = APPLY ? p.Nvalid : p.z.ld;   // multiples of 4 on these paths
      const int cbase = nt * BN + half * (BN / 2) + lq * 4;
      // The old W does not depend on the MMAs: while this tile's accumulator is still being produced,
      // pull the first block of W into registers and ask L2 for the rest of the tile.
      float4 wv[8];
#pragma unroll
      for (int g = 0; g < 8; ++g) wv[g] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (APPLY) {
#pragma unroll
        for (int g = 0; g < 8; ++g)
          if (rowp[g] != nullptr && cbase < ncols) wv[g] = __ldcs(reinterpret_cast<const float4*>(rowp[g] + cbase));
        if (lq == 0) {   // one 128-byte line per (row, 32-column block)
#pragma unroll
          for (int g = 0; g < 8; ++g)
            for (int cc = 1; cc < BN / 64; ++cc)
              if (rowp[g] != nullptr && cbase + cc * 32 < ncols)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(rowp[g] + cbase + cc * 32));
        }
      }
      ok = wait_or_abort(&ctl->tmem_full[buf], acc_ph, ctl, p.status);
      if (!ok) break;
      ptx::tc_fence_after();
      const uint32_t taddr = tmem_base + buf * ACC_COLS + ((uint32_t)(quarter * 32) << 16);
      if (!APPLY && EPI == 1) {
        // ---- multiclass-logistic epilogue: thread = sample row while the values sit in registers
        const float kLog2e = 1.4426950408889634f;
        const int ccol0 = nt * BN + half * (BN / 2);     // first class of this warp's half tile
        float m = -INFINITY;
#pragma unroll 1
        for (int cc = 0; cc < BN / 64; ++cc) {
          uint32_t v[32];
          ptx::tmem_ld32(taddr + half * (BN / 2) + cc * 32, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 32; ++q)
            if (ccol0 + cc * 32 + q < p.Nvalid) m = fmaxf(m, __uint_as_float(v[q]));
        }
        const float mb = (m == -INFINITY) ? 0.f : m * kLog2e;   // half tile entirely beyond the last class
        float ssum = 0.f;
#pragma unroll 1
        for (int cc = 0; cc < BN / 64; ++cc) {
          const int c = cbase + cc * 32;
          uint32_t v[32];
          ptx::tmem_ld32(taddr + half * (BN / 2) + cc * 32, v);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 32; ++q) {
            const float ex = (ccol0 + cc * 32 + q < p.Nvalid) ? exp2f(fmaf(__uint_as_float(v[q]), kLog2e, -mb)) : 0.f;
            ssum += ex;
            v[q] = __float_as_uint(ex);
          }
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<uint4*>(stage + lane * 32 + ((q ^ (lane & 7)) << 2)) =
                make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          __syncwarp();
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const int lr = 4 * g + lrow;
            const float4 a = *reinterpret_cast<const float4*>(stage + lr * 32 + ((lq ^ (lr & 7)) << 2));
            if (rowp[g] != nullptr && c < ncols) {
              if (p.z.es == 4) {
                __stcs(reinterpret_cast<float4*>(rowp[g] + c), a);
              } else {
                __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                __stcs(reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(rowp[g]) + c), pk);
              }
            }
          }
          __syncwarp();
        }
        {   // (max, sum) of this thread's own row
          const int r = quarter * 32 + lane;
          int wp_, slot;
          if (p.B >= BM) { wp_ = mt / p.m_tpw; slot = (mt % p.m_tpw) * BM + r; }
          else { wp_ = mt * p.m_wp + r / p.m_bb; slot = r % p.m_bb; }
          if (wp_ < p.P && slot < p.B)
            p.stats[(long long)(wp_ * p.B + slot) * p.n_parts + nt * 2 + half] = make_float2(m, ssum);
        }
      } else
#pragma unroll 1
      for (int cc = 0; cc < BN / 64; ++cc) {
        const int col_in_tile = half * (BN / 2) + cc * 32;
        const int c = cbase + cc * 32;
        uint32_t v[32];
        ptx::tmem_ld32(taddr + col_in_tile, v);
        float4 wn[8];   // next block of W, in flight while this block is combined and stored
#pragma unroll
        for (int g = 0; g < 8; ++g) wn[g] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (APPLY && cc + 1 < BN / 64) {
#pragma unroll
          for (int g = 0; g < 8; ++g)
            if (rowp[g] != nullptr && c + 32 < ncols) wn[g] = __ldcs(reinterpret_cast<const float4*>(rowp[g] + c + 32));
        }
        ptx::tmem_ld_wait();
        if (SPLIT) {   // main accumulator + correction accumulator, one fp32 addition (round to nearest) per value
          uint32_t lo[32];
          ptx::tmem_ld32(taddr + BN + col_in_tile, lo);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 32; ++q) v[q] = __float_as_uint(__uint_as_float(v[q]) + __uint_as_float(lo[q]));
        }
        if (cc == BN / 64 - 1) {   // the last of this warp's accumulator columns are in registers: the MMAs may go on
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (CG == 1 || rank == 0) ptx::mbar_arrive(&ctl->tmem_empty[buf]);
            else ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[buf]), 0));
          }
        }
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(stage + lane * 32 + ((q ^ (lane & 7)) << 2)) =
              make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        __syncwarp();
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const int lr = 4 * g + lrow;
          const float4 a = *reinterpret_cast<const float4*>(stage + lr * 32 + ((lq ^ (lr & 7)) << 2));
          if (rowp[g] != nullptr && c < ncols) {
            if (APPLY) {
              float4 w = wv[g];
              w.x = fmaf(-p.eta, a.x, w.x); w.y = fmaf(-p.eta, a.y, w.y);
              w.z = fmaf(-p.eta, a.z, w.z); w.w = fmaf(-p.eta, a.w, w.w);
              // the new fp32 W goes out by a TMA bulk store of the whole staging block (below): fewer store
              // instructions than per-thread 16-byte stores
              *reinterpret_cast<float4*>(stage + lr * 32 + ((lq ^ (lr & 7)) << 2)) = w;
              if (SPLIT && p.shadow != nullptr) {
                // the correction operand of the new W (B side: values, then remainders of what the tensor core sees)
                const float rx = w.x - __uint_as_float(__float_as_uint(w.x) & 0xFFFFE000u);
                const float ry = w.y - __uint_as_float(__float_as_uint(w.y) & 0xFFFFE000u);
                const float rz = w.z - __uint_as_float(__float_as_uint(w.z) & 0xFFFFE000u);
                const float rw = w.w - __uint_as_float(__float_as_uint(w.w) & 0xFFFFE000u);
                __nv_bfloat162 v0 = __floats2bfloat162_rn(w.x, w.y), v1 = __floats2bfloat162_rn(w.z, w.w);
                __nv_bfloat162 r0 = __floats2bfloat162_rn(rx, ry), r1 = __floats2bfloat162_rn(rz, rw);
                const long long j = mt * BM + quarter * 32 + lr;
                uint2* dst = reinterpret_cast<uint2*>(p.shadow + (j * p.w_atoms + (c >> 5)) * 64 + (c & 31));
                __stcs(dst, make_uint2(*reinterpret_cast<uint32_t*>(&v0), *reinterpret_cast<uint32_t*>(&v1)));
                __stcs(dst + 8, make_uint2(*reinterpret_cast<uint32_t*>(&r0), *reinterpret_cast<uint32_t*>(&r1)));
              } else if (p.shadow != nullptr) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                __stcs(reinterpret_cast<uint2*>(p.shadow + (rowp[g] - p.W) + c), pk);
              }
            } else {
              __stcs(reinterpret_cast<float4*>(rowp[g] + c), a);
            }
          }
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) wv[g] = wn[g];
        if (APPLY) {   // the 32 x 32 block of new W sits in the staging block, swizzled as the tensor map expects
          ptx::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            ptx::tma_store_2d(&tmW, stage, nt * BN + col_in_tile, mt * BM + quarter * 32);
            ptx::tma_store_commit();
            ptx::tma_store_wait_read();   // the block is rewritten by the next pass
          }
        }
        __syncwarp();
      }
      if (!APPLY && EPI == 1) {   // (the other epilogues signal from inside their last block)
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {   // this warp's part of the accumulator is drained
          if (CG == 1 || rank == 0) ptx::mbar_arrive(&ctl->tmem_empty[buf]);
          else ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&ctl->tmem_empty[buf]), 0));
        }
      }
    }
  }

  if (APPLY && warp >= 2 && lane == 0) ptx::tma_store_wait_all();
  ptx::tc_fence_before();
  __syncthreads();
  if (CG == 2) ptx::cluster_sync();   // nobody leaves while its pair may still signal it or read its tiles
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc<CG>(tmem_base, NBUF * ACC_COLS);
  }
}

// ------------------------------------------------------------------------------------------- host side
PFN_cuTensorMapEncodeTiled_v12000 get_encode() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (fn == nullptr) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(ptr);
  }
  return fn;
}

// Tensor map over factor-like rows (row r of worker w at base + w * worker_stride + r * row_stride).
//   fold == false: 3-D (value, row, worker); box = {CH values, box_rows, box_workers}.
//   fold == true : 4-D (value within a 128-byte chunk, row, worker, chunk) with the chunk dimension
//                  striding 128 bytes along the row; box = {CH, box_rows, box_workers, box_chunks}.
//                  `cols` must be a multiple of CH (a chunk never straddles the end of a row).
bool encode_rows_map(CUtensorMap* m, int es, const void* base, long long cols, long long rows, long long workers,
                     long long row_stride_bytes, long long worker_stride_bytes, int box_rows, int box_workers,
                     bool fold, int box_chunks, bool atom32) {
  auto fn = get_encode();
  if (fn == nullptr) return false;
  const int CH = 128 / es;
  const CUtensorMapDataType dt = es == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
  const CUtensorMapSwizzle sw = atom32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B;
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r;
  if (!fold) {
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)workers};
    cuuint64_t strides[2] = {(cuuint64_t)row_stride_bytes, (cuuint64_t)worker_stride_bytes};
    cuuint32_t box[3] = {(cuuint32_t)CH, (cuuint32_t)box_rows, (cuuint32_t)box_workers};
    r = fn(m, dt, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    // whole chunks; a caller that folds a row length that is no multiple of CH (the u rows of the apply) gets
    // the tail of the last chunk from the bytes that follow the row, and must discard those output indices
    cuuint64_t dims[4] = {(cuuint64_t)CH, (cuuint64_t)rows, (cuuint64_t)workers, (cuuint64_t)((cols + CH - 1) / CH)};
    cuuint64_t strides[3] = {(cuuint64_t)row_stride_bytes, (cuuint64_t)worker_stride_bytes, 128};
    cuuint32_t box[4] = {(cuuint32_t)CH, (cuuint32_t)box_rows, (cuuint32_t)box_workers, (cuuint32_t)box_chunks};
    r = fn(m, dt, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  return r == CUDA_SUCCESS;
}

int pow2_at_least(int n) {
  int p = 1;
  while (p < n) p <<= 1;
  return p;
}

template <int ES, bool APPLY, int BN, int CG, int KA, bool FOLD, int EPI, bool SPLIT = false>
int launch_gemm(cudaStream_t s, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& w, const CUtensorMap& ac,
                const CUtensorMap& bc, const GemmParams& p, int num_sms) {
  constexpr int stage_bytes = (BM + BN / CG) * 128 * KA * (SPLIT ? 2 : 1);
  constexpr int threads = NUM_THREADS;
  constexpr int stages = (RING_BYTES / stage_bytes) < MAX_STAGES ? (RING_BYTES / stage_bytes) : MAX_STAGES;
  constexpr int smem = stages * stage_bytes + EPI_STAGE_BYTES + 1024 + (int)sizeof(SharedCtl);
  auto kernel = umma_gemm_kernel<ES, APPLY, BN, CG, KA, FOLD, EPI, SPLIT>;
  static PerDeviceOnce attr_once;   // function attributes are per device
  static int max_clusters = 0;
  if (attr_once.first()) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
      return SFB_ERR_CUDA;
    if (CG == 2) {   // how many CTA pairs the device can hold at once
      cudaLaunchConfig_t q;
      memset(&q, 0, sizeof(q));
      cudaLaunchAttribute qa[1];
      qa[0].id = cudaLaunchAttributeClusterDimension;
      qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
      q.gridDim = dim3(num_sms & ~1, 1, 1);
      q.blockDim = dim3(threads, 1, 1);
      q.dynamicSmemBytes = smem;
      q.attrs = qa; q.numAttrs = 1;
      if (cudaOccupancyMaxActiveClusters(&max_clusters, kernel, &q) != cudaSuccess || max_clusters < 1) {
        cudaGetLastError();
        max_clusters = num_sms / 2;
      }
    }
  }
  const int tiles = p.m_tiles * p.n_tiles * p.k_splits;
  if (CG == 1) {
    const int grid = tiles < num_sms ? tiles : num_sms;
    kernel<<<grid, threads, smem, s>>>(a, b, w, ac, bc, p);
  } else {
    const int clusters = tiles < max_clusters ? tiles : max_clusters;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(2 * clusters, 1, 1);
    cfg.blockDim = dim3(threads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = at; cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, a, b, w, ac, bc, p) != cudaSuccess) return SFB_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? 1 : SFB_ERR_CUDA;
}

// Kernel variants: "big" = CTA pairs on 256 x 256 tiles; with J, D multiples of the chunk it also folds
// the operand loads (one TMA per operand per stage) and doubles the reduction depth of a stage.
struct Variant {
  int bn, cg, ka;
  bool fold;
  bool split;   // error-compensated tf32: 128-column tiles, one atom per stage, lo tiles made in shared memory
};

// ac / bc: tensor maps of the correction operands (compensated kernels only; the others get the plain maps again)
template <int ES, bool APPLY, int EPI>
int dispatch_es(cudaStream_t s, const Variant& v, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& w,
                const CUtensorMap& ac, const CUtensorMap& bc, const GemmParams& p, int num_sms) {
  if (v.split) {
    if (ES == 4 && EPI == 0) {   // the only instantiations: fp32 operands, plain stores / W write-back
      if (v.cg == 2 && v.bn == 256 && v.fold) return launch_gemm<4, APPLY, 256, 2, 1, true, 0, true>(s, a, b, w, ac, bc, p, num_sms);
      if (v.cg == 2 && v.bn == 256) return launch_gemm<4, APPLY, 256, 2, 1, false, 0, true>(s, a, b, w, ac, bc, p, num_sms);
      if (v.cg == 2 && v.fold) return launch_gemm<4, APPLY, 128, 2, 1, true, 0, true>(s, a, b, w, ac, bc, p, num_sms);
      if (v.cg == 2) return launch_gemm<4, APPLY, 128, 2, 1, false, 0, true>(s, a, b, w, ac, bc, p, num_sms);
      return launch_gemm<4, APPLY, 128, 1, 1, false, 0, true>(s, a, b, w, ac, bc, p, num_sms);
    }
    return SFB_ERR_UNSUPPORTED;
  }
  if (v.cg == 2) {
    if (v.fold && v.ka == 2) return launch_gemm<ES, APPLY, 256, 2, 2, true, EPI>(s, a, b, w, a, b, p, num_sms);
    if (v.fold) return launch_gemm<ES, APPLY, 256, 2, 1, true, EPI>(s, a, b, w, a, b, p, num_sms);
    if (v.ka == 2) return launch_gemm<ES, APPLY, 256, 2, 2, false, EPI>(s, a, b, w, a, b, p, num_sms);
    return launch_gemm<ES, APPLY, 256, 2, 1, false, EPI>(s, a, b, w, a, b, p, num_sms);
  }
  if (v.bn == 256) return launch_gemm<ES, APPLY, 256, 1, 1, false, EPI>(s, a, b, w, a, b, p, num_sms);
  if (v.ka == 2) return launch_gemm<ES, APPLY, 128, 1, 2, false, EPI>(s, a, b, w, a, b, p, num_sms);
  return launch_gemm<ES, APPLY, 128, 1, 1, false, EPI>(s, a, b, w, a, b, p, num_sms);
}

template <bool APPLY, int EPI>
int dispatch_gemm(cudaStream_t s, int es, const Variant& v, const CUtensorMap& a, const CUtensorMap& b,
                  const CUtensorMap& w, const CUtensorMap& ac, const CUtensorMap& bc, const GemmParams& p, int num_sms) {
  return es == 2 ? dispatch_es<2, APPLY, EPI>(s, v, a, b, w, ac, bc, p, num_sms)
                 : dispatch_es<4, APPLY, EPI>(s, v, a, b, w, ac, bc, p, num_sms);
}

// Tensor maps of the correction operands (bf16, 128-byte swizzle, always whole 128-byte atoms).
// K-major: dst[row][atom][64] as (value, row, worker, atom), rows of all workers consecutive.
bool encode_corr_k_map(CUtensorMap* m, const void* base, long long rows_per_worker, long long workers, long long atoms,
                       int box_rows, int box_workers) {
  auto fn = get_encode();
  if (fn == nullptr) return false;
  cuuint64_t dims[4] = {64, (cuuint64_t)rows_per_worker, (cuuint64_t)workers, (cuuint64_t)atoms};
  cuuint64_t strides[3] = {(cuuint64_t)atoms * 128, (cuuint64_t)rows_per_worker * atoms * 128, 128};
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_workers, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// MN-major: dst[line][ldc] as (value within a chunk of 64, line, chunk); a box is 64 lines of box_chunks chunks.
bool encode_corr_mn_map(CUtensorMap* m, const void* base, long long ldc, long long lines, int box_chunks) {
  auto fn = get_encode();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {64, (cuuint64_t)lines, (cuuint64_t)(ldc / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)ldc * 2, 128};
  cuuint32_t box[3] = {64, 64, (cuuint32_t)box_chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

constexpr int MAX_SPLITS = 8;   // ranges a forward reduction may be cut into (partial buffers of the plan)
constexpr int X3_MAX_SPLITS = 32;   // ... on the compensated path, where the count is also tuned to fill whole waves

struct UmmaPlan {
  sfb_desc d;
  Layout l;
  int num_sms;
  int es;
  int max_splits; // ranges a forward reduction may be cut into = partial buffers allocated
  bool x3;        // error-compensated tf32 (SFB_PATH_TF32X3): the SPLIT kernels, forward always through partial buffers
  float2* stats;  // MLR: (max, sum of exps) per (sample, half tile) from the forward GEMM's epilogue
  // compensated kernels: correction operands of the sample rows (forward) and of the factor rows (apply),
  // rewritten by a pre-pass before every GEMM launch
  void* xc;
  void* uc;
  void* vc;
  int ldcu, ldcv;               // padded row lengths (multiples of 64) of uc / vc
  // Set by a factor stage that wrote uc / vc itself, beside the factors (its finishing pass, its copy of v): the
  // rows they were made from and how many pairs.  The next apply of exactly those rows skips its pre-pass; any
  // other call clears them.
  const void* fresh_u;
  const void* fresh_v;
  int fresh_K;
  float* part_ws;               // partial products of a split reduction, [MAX_SPLITS][K][ldp] fp32 (small forward GEMMs only)
  int ldp;
  // MLR: the factor v is a copy of x that nothing in the factor stage reads, so it runs on a side stream
  // next to the forward GEMM (fork / join by events)
  cudaStream_t side;
  cudaEvent_t fork, join;
  bool side_ok;
  // Test hook.  SFB_TEST_LOSE_SIGNAL=1 in the environment at plan creation: the first GEMM launched through this
  // plan loses one pipeline signal in its first CTA (pair), which must end in SFB_DEV_TIMEOUT after the bounded
  // wait, not in a hang.  The only environment variable the library reads.
  int lose_signal;
};

// Tile order: tiles of the fast dimension walked before the slow one advances.  Eight 256-wide column tiles keep
// the slab of the smaller factor matrix (64 MB of V at 32768 x 8192, K = 4096, bf16) in L2 while the other streams.
constexpr int FWD_GROUP = 8, APPLY_GROUP = 8;
// 128-byte atoms of the reduction index per pipeline stage wherever three such stages fit in shared memory.
constexpr int STAGE_ATOMS = 2;
// Compensated kernels: 128-byte atoms (32 fp32 reduction steps = 4 MMA instructions) one accumulator may take
// before its range ends: 40 atoms = 160 roundings toward zero, about 2.6e-6 of the sum.
constexpr int X3_ATOMS_PER_RANGE = 40;
// ... and pairs one launch of the compensated apply takes (128 instructions: 2e-6 of the sum; measured: 4096 pairs in
// one launch come out at 1.0e-5, 2048 at 5e-6); larger updates are applied in several launches.
constexpr int X3_PAIRS_PER_APPLY = 1024;

int umma_plan_create(const sfb_desc& d, const Layout& l, UmmaPlan** out) {
  if (get_encode() == nullptr) return SFB_ERR_CUDA;
  UmmaPlan* p = new UmmaPlan();
  p->d = d; p->l = l;
  p->es = (d.path == SFB_PATH_BF16) ? 2 : 4;
  p->x3 = d.path == SFB_PATH_TF32X3;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&p->num_sms, cudaDevAttrMultiProcessorCount, dev);
  const char* ls = getenv("SFB_TEST_LOSE_SIGNAL");
  p->lose_signal = (ls != nullptr && ls[0] == '1') ? 1 : 0;
  p->part_ws = nullptr;
  p->xc = p->uc = p->vc = nullptr;
  p->fresh_u = p->fresh_v = nullptr;
  p->fresh_K = 0;
  p->ldcu = (int)pad_to(d.J, 64);
  p->ldcv = (int)pad_to(d.D, 64);
  p->ldp = (int)pad_to(d.J, 4);
  {   // forward GEMMs whose 128 x 128 tiles do not fill the SMs may split their reduction
    const long long K_ = (long long)d.P * d.B;
    const long long tiles = ((K_ + 127) / 128) * ((d.J + 127) / 128);
    // the compensated path tunes the count up to 16, within 4 GB of partial buffers
    p->max_splits = MAX_SPLITS;
    if (p->x3) {
      const long long one = K_ * p->ldp * 4;
      long long n = (4LL << 30) / (one > 0 ? one : 1);
      p->max_splits = (int)(n < 1 ? 1 : (n > X3_MAX_SPLITS ? X3_MAX_SPLITS : n));
    }
    if ((tiles < p->num_sms || p->x3) && cudaMalloc(&p->part_ws, (size_t)p->max_splits * K_ * p->ldp * 4) != cudaSuccess) {
      cudaGetLastError();
      delete p;
      return SFB_ERR_ALLOC;
    }
  }
  if (p->x3) {
    const size_t K_ = (size_t)d.P * d.B;
    // reduction blocks of 32 pairs as the apply takes them: whole blocks per worker, or several workers per block
    const size_t blocks = d.B >= 32 ? (size_t)d.P * ((d.B + 31) / 32) : ((size_t)d.P + 32 / pow2_at_least(d.B) - 1) / (32 / pow2_at_least(d.B));
    // zeroed once: what no writer touches (columns beyond a row's padded length, lines of rows that do not exist,
    // the tail of a row's last atom) must read as zeros, as the fp32 operands' out-of-range elements do
    const bool ok = cudaMalloc(&p->xc, K_ * ((d.D + 31) / 32) * 128) == cudaSuccess &&
                    cudaMalloc(&p->uc, blocks * 64 * p->ldcu * 2) == cudaSuccess &&
                    cudaMalloc(&p->vc, blocks * 64 * p->ldcv * 2) == cudaSuccess &&
                    cudaMemset(p->xc, 0, K_ * ((d.D + 31) / 32) * 128) == cudaSuccess &&
                    cudaMemset(p->uc, 0, blocks * 64 * p->ldcu * 2) == cudaSuccess &&
                    cudaMemset(p->vc, 0, blocks * 64 * p->ldcv * 2) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      if (p->xc) cudaFree(p->xc);
      if (p->uc) cudaFree(p->uc);
      if (p->vc) cudaFree(p->vc);
      if (p->part_ws) cudaFree(p->part_ws);
      delete p;
      return SFB_ERR_ALLOC;
    }
  }
  p->side_ok = false;
  {
    if (d.model == SFB_MLR) {
      p->side_ok = cudaStreamCreateWithFlags(&p->side, cudaStreamNonBlocking) == cudaSuccess;
      if (p->side_ok) {
        const bool e1 = cudaEventCreateWithFlags(&p->fork, cudaEventDisableTiming) == cudaSuccess;
        const bool e2 = e1 && cudaEventCreateWithFlags(&p->join, cudaEventDisableTiming) == cudaSuccess;
        if (!e2) {
          if (e1) cudaEventDestroy(p->fork);
          cudaStreamDestroy(p->side);
          cudaGetLastError();
          p->side_ok = false;
        }
      }
    }
  }
  p->stats = nullptr;
  if (d.model == SFB_MLR) {
    const size_t parts = 2 * (size_t)((d.J + 127) / 128);
    if (cudaMalloc(&p->stats, (size_t)d.P * d.B * parts * sizeof(float2)) != cudaSuccess) {
      cudaGetLastError();
      if (p->part_ws) cudaFree(p->part_ws);
      if (p->xc) cudaFree(p->xc);
      if (p->uc) cudaFree(p->uc);
      if (p->vc) cudaFree(p->vc);
      delete p;
      return SFB_ERR_ALLOC;
    }
  }
  *out = p;
  return SFB_OK;
}

void umma_plan_destroy(UmmaPlan* p) {
  if (p->side_ok) {
    cudaStreamSynchronize(p->side);
    cudaEventDestroy(p->fork);
    cudaEventDestroy(p->join);
    cudaStreamDestroy(p->side);
  }
  if (p->stats) cudaFree(p->stats);
  if (p->part_ws) cudaFree(p->part_ws);
  if (p->xc) cudaFree(p->xc);
  if (p->uc) cudaFree(p->uc);
  if (p->vc) cudaFree(p->vc);
  delete p;
}

// Tile shape and kernel variant for an M x N output (M counted in 128-row units).
// max_splits > 1: the caller can take partial products, so a problem with few tiles may cut its reduction
// (k_atoms 128-byte atoms long) into *splits ranges.  CTA pairs on 256 x 256 tiles need half the operand
// traffic per flop of single 128 x 128 tiles, so they are preferred as soon as pairs x ranges fill the SMs.
static Variant pick_variant(const UmmaPlan* pl, int m_units, int N, bool dims_chunk_aligned, int k_atoms = 0,
                            int max_splits = 1, int* splits = nullptr) {
  Variant v;
  v.split = false;
  if (splits != nullptr) *splits = 1;
  if (pl->x3) {
    // Compensated kernels: one atom of the reduction per stage (fp32 tiles and their bf16 correction tiles).  These
    // kernels run at the rate L2 delivers their operands, so a candidate shape costs the bytes its busiest SM loads:
    //   256 x 128 pair tiles: 48 KB per stage and CTA; the accumulators (main, corrections) of two tiles fill the
    //     512 columns of tensor memory, so a tile's epilogue overlaps the MMAs of the next;
    //   256 x 256 pair tiles: 64 KB per stage for twice the work, but one accumulator set: the epilogue is exposed
    //     (about 8 stages' worth per tile, measured at 4096 x 10000, K = 1024);
    //   128 x 128 single tiles (64 KB per stage): for a single row unit, or when an odd number of row units would
    //     leave the last pair half empty and waves of singles are shorter (an apply of 600 rows).
    // With a split reduction (forward; ranges added in fp32 by the finishing pass) the number of ranges is chosen
    // with the shape: enough of them that one accumulator takes at most X3_ATOMS_PER_RANGE atoms (every instruction
    // rounds the sum toward zero, about 1.6e-8 of it), and the count with the least cost among the admissible ones
    // (a little is added per range for its partial buffer).
    v.split = true;
    v.ka = 1;
    const bool ranged = splits != nullptr && k_atoms > 0 && max_splits > 1;
    const long long k_len = k_atoms > 0 ? k_atoms : 32;          // atoms of the reduction (apply: 32 pairs each)
    long long best_cost = -1;
    auto consider = [&](int bn, int cg) {
      const long long stage_kb = (BM + bn / cg) * 256 / 1024;    // fp32 + correction tiles of one CTA
      const long long epi = (4 * bn > 512) ? 8 * stage_kb : 0;   // exposed epilogue, in KB loaded
      const long long tiles = (long long)((m_units + cg - 1) / cg) * ((N + bn - 1) / bn);
      const long long slots = pl->num_sms / cg;
      long long ks_lo = 1, ks_hi = 1;
      if (ranged) {
        ks_lo = (k_len + X3_ATOMS_PER_RANGE - 1) / X3_ATOMS_PER_RANGE;
        if (ks_lo > max_splits) ks_lo = max_splits;
        if (ks_lo < 1) ks_lo = 1;
        ks_hi = max_splits;
      }
      for (long long ks = ks_lo; ks <= ks_hi && (ks == ks_lo || k_len >= 4 * ks); ++ks) {
        const long long per = (k_len + ks - 1) / ks;
        const long long n_ranges = (k_len + per - 1) / per;          // ranges that exist
        const long long waves = (tiles * n_ranges + slots - 1) / slots;
        const long long cost = waves * (per * stage_kb + epi) + (ranged ? n_ranges * stage_kb * 3 / 8 : 0);
        if (best_cost < 0 || cost < best_cost) {
          best_cost = cost;
          v.bn = bn; v.cg = cg;
          if (splits != nullptr) *splits = (int)ks;
        }
      }
    };
    if (m_units >= 2) {
      consider(128, 2);
      if (N > 128) consider(256, 2);
      if ((m_units & 1) && !ranged) consider(128, 1);
    } else {
      consider(128, 1);
    }
    v.fold = v.cg == 2 && dims_chunk_aligned;
    return v;
  }
  v.bn = (N > 128 && (long long)m_units * ((N + 255) / 256) >= pl->num_sms) ? 256 : 128;
  // CTA pairs (256-row tiles) once there is enough work to fill the machine with them
  v.cg = (v.bn == 256 && (long long)((m_units + 1) / 2) * ((N + 255) / 256) >= pl->num_sms / 2) ? 2 : 1;
  if (v.cg == 1 && k_atoms > 0) {
    const int k_blocks = (k_atoms + STAGE_ATOMS - 1) / STAGE_ATOMS;
    auto ranges = [&](long long tiles, int slots) {
      long long ks = slots / (tiles > 0 ? tiles : 1);
      if (ks > max_splits) ks = max_splits;
      while (ks > 1 && k_blocks < 16 * ks) --ks;
      return (int)(ks < 1 ? 1 : ks);
    };
    const long long t_pair = (long long)((m_units + 1) / 2) * ((N + 255) / 256);
    const int ks_pair = ranges(t_pair, pl->num_sms / 2);
    const long long t_one = (long long)m_units * ((N + 127) / 128);
    const int ks_one = ranges(t_one, pl->num_sms);
    // pairs that fill three quarters of the machine beat single tiles that fill all of it: the single
    // 128 x 128 tiles are bound by the operand feed (about 50 % tensor-pipe activity with fp32 operands)
    if (N > 128 && m_units >= 2 && 4 * t_pair * ks_pair >= 3 * (pl->num_sms / 2)) {
      v.bn = 256; v.cg = 2;
      if (splits != nullptr) *splits = ks_pair;
    } else if (t_one < pl->num_sms && splits != nullptr && max_splits > 1) {
      v.bn = 128; v.cg = 1;
      *splits = ks_one;
    }
  }
  v.fold = v.cg == 2 && dims_chunk_aligned;
  // two 128-byte atoms of reduction per stage wherever three such stages fit in shared memory: the
  // per-stage barrier round trip, not the number of TMA instructions, is what costs
  v.ka = (v.cg == 2 || v.bn == 128) ? STAGE_ATOMS : 1;
  return v;
}

// Z rows (fp32, through `z`) = A rows (through `a`, the path's value type) times W^T.
int umma_forward_rows(UmmaPlan* pl, cudaStream_t s, const void* Wop, RowMap a, RowMap z, int* dev_status,
                      float2* stats, int* n_parts_out, int* part_cols_out, int* k_splits_out, int max_splits,
                      long long split_stride, int workers, const void* w_corr, bool a_corr_ready) {
  const sfb_desc& d = pl->d;
  const int es = pl->es, CH = 128 / es;
  const int P = workers > 0 ? workers : d.P;     // a shard of the workers, or all of them
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.B = d.B; p.P = P;
  int m_units;
  if (d.B >= BM) { p.m_bb = BM; p.m_wp = 1; p.m_tpw = (d.B + BM - 1) / BM; m_units = P * p.m_tpw; }
  else { p.m_bb = pow2_at_least(d.B); p.m_wp = BM / p.m_bb; p.m_tpw = 1; m_units = (P + p.m_wp - 1) / p.m_wp; }
  // folding walks the reduction index (D) in 128-byte atoms: rows must be whole atoms long
  const bool may_split = k_splits_out != nullptr && stats == nullptr && max_splits > 1;
  int ks_pick = 1;
  const Variant v = pick_variant(pl, m_units, d.J, (d.D % CH) == 0 && (a.ld % CH) == 0, (d.D + CH - 1) / CH,
                                 may_split ? (max_splits < pl->max_splits ? max_splits : pl->max_splits) : 1, &ks_pick);
  p.m_tiles = (m_units + v.cg - 1) / v.cg;
  p.n_tiles = (d.J + v.bn - 1) / v.bn;
  p.k_blocks = (d.D + CH * v.ka - 1) / (CH * v.ka);
  // Few tiles and a long reduction (e.g. 1024 samples x 1000 classes over 20000 features): cut the
  // reduction so that every SM gets work; the partial products are summed, in a fixed order, by the
  // finishing pass.  Only when the caller provides the partial buffers (k_splits_out != nullptr).
  p.k_splits = may_split ? ks_pick : 1;
  if (k_splits_out != nullptr) *k_splits_out = p.k_splits;
  p.k_per_split = (p.k_blocks + p.k_splits - 1) / p.k_splits;
  // no empty range: a work item without reduction blocks would never signal its accumulator (and the finishing pass
  // would add a partial buffer nobody wrote)
  p.k_splits = (p.k_blocks + p.k_per_split - 1) / p.k_per_split;
  if (k_splits_out != nullptr) *k_splits_out = p.k_splits;
  p.split_stride = split_stride;
  // the operand that does not fit in L2 should stream from HBM once: consecutive tiles share its slab
  p.m_fastest = ((long long)d.J * d.D > (long long)P * d.B * d.D) ? 1 : 0;
  p.a_policy = p.m_fastest ? 2 : 0;   // the operand whose slab changes every tile is re-read all along: keep it
  p.b_policy = p.m_fastest ? 0 : 2;
  p.group = FWD_GROUP;
  p.z = z;
  p.status = dev_status;
  p.lose_signal = pl->lose_signal;
  pl->lose_signal = 0;
  p.Nvalid = d.J;
  p.stats = stats;
  p.n_parts = 2 * p.n_tiles;
  if (n_parts_out != nullptr) *n_parts_out = p.n_parts;
  if (part_cols_out != nullptr) *part_cols_out = v.bn / 2;
  CUtensorMap ta, tb;
  if (!encode_rows_map(&ta, es, a.base, d.D, d.B, P, (long long)a.ld * es, a.worker_stride, p.m_bb, p.m_wp, v.fold,
                       v.ka, false))
    return SFB_ERR_CUDA;
  if (!encode_rows_map(&tb, es, Wop, d.D, d.J, 1, (long long)d.D * es, (long long)d.D * es * d.J, v.bn / v.cg, 1,
                       v.fold, v.ka, false))
    return SFB_ERR_CUDA;
  CUtensorMap tac = ta, tbc = tb;
  int launches = 0;
  if (pl->x3) {
    // correction operands: the sample rows' are written here, W's come from the caller (it knows when W changed)
    if (w_corr == nullptr) return SFB_ERR_ARG;
    const int atoms = (d.D + 31) / 32;
    if (!a_corr_ready) {   // (the kernel that made the rows may have written their correction operand with them)
      const int r = launch_split_k(s, a, P * d.B, d.D, pl->xc, true);
      if (r < 0) return r;
      launches += r;
    }
    if (!encode_corr_k_map(&tac, pl->xc, d.B, P, atoms, p.m_bb, p.m_wp) ||
        !encode_corr_k_map(&tbc, w_corr, d.J, 1, atoms, v.bn / v.cg, 1))
      return SFB_ERR_CUDA;
  }
  const int r = stats != nullptr ? dispatch_gemm<false, 1>(s, es, v, ta, tb, ta, tac, tbc, p, pl->num_sms)
                                 : dispatch_gemm<false, 0>(s, es, v, ta, tb, ta, tac, tbc, p, pl->num_sms);
  return r < 0 ? r : launches + r;
}

// Sparse coding on the tensor cores: u rows = dense code rows `a` times W^T, minus the data rows.
// Geometry of the apply's reduction blocks (32 pairs each) for a kernel that writes a correction operand.
static CorrOut apply_corr(const UmmaPlan* pl, void* dst, int ldc, bool a_side) {
  CorrOut c;
  c.mn = reinterpret_cast<char*>(dst);
  c.ldc = ldc;
  c.a_side = a_side ? 1 : 0;
  const int B = pl->d.B;
  if (B >= 32) { c.k_bb = 32; c.k_wp = 1; c.k_bpw = (B + 31) / 32; }
  else { c.k_bb = pow2_at_least(B); c.k_wp = 32 / c.k_bb; c.k_bpw = 1; }
  return c;
}

CorrOut umma_codes_corr(UmmaPlan* pl, bool for_apply) {
  if (!pl->x3) return CorrOut();
  CorrOut c = for_apply ? apply_corr(pl, pl->vc, pl->ldcv, false) : CorrOut();
  c.km = reinterpret_cast<char*>(pl->xc);
  c.atoms = (pl->d.D + 31) / 32;
  return c;
}

int umma_forward_sc(UmmaPlan* pl, cudaStream_t s, const void* W, RowMap a, RowMap u, const float* Xdata, int* dev_status,
                    int workers, const void* w_corr, bool for_apply, const CorrOut* a_corr) {
  const sfb_desc& d = pl->d;
  const int K = (workers > 0 ? workers : d.P) * d.B;
  int r, launches = 0;
  pl->fresh_u = pl->fresh_v = nullptr;
  pl->fresh_K = 0;
  const bool emit = pl->x3 && for_apply && workers == 0;
  const CorrOut cu = emit ? apply_corr(pl, pl->uc, pl->ldcu, true) : CorrOut();
  // the kernel that made the code rows wrote their correction operands: the forward's, and perhaps the apply's
  const bool a_ready = pl->x3 && a_corr != nullptr && a_corr->km == reinterpret_cast<char*>(pl->xc);
  const void* v_fresh = (emit && a_corr != nullptr && a_corr->mn == reinterpret_cast<char*>(pl->vc)) ? a.base : nullptr;
  if (pl->part_ws != nullptr) {   // reduction in ranges (few tiles, or the compensated path): summed by the finishing pass
    RowMap pz;
    pz.base = reinterpret_cast<char*>(pl->part_ws); pz.ld = pl->ldp; pz.B = d.B; pz.es = 4;
    pz.worker_stride = (long long)d.B * pl->ldp * 4;
    const long long sstride = (long long)d.P * d.B * pl->ldp * 4;
    int ks = 1;
    if ((r = umma_forward_rows(pl, s, W, a, pz, dev_status, nullptr, nullptr, nullptr, &ks, pl->max_splits, sstride, workers,
                               w_corr, a_ready)) < 0)
      return r;
    launches += r;
    if ((r = launch_finish_sc(s, pz, u, Xdata, K, d.J, ks, sstride, cu)) < 0) return r;
    if (emit) { pl->fresh_u = u.base; pl->fresh_v = v_fresh; pl->fresh_K = K; }
    return launches + r;
  }
  if ((r = umma_forward_rows(pl, s, W, a, u, dev_status, nullptr, nullptr, nullptr, nullptr, 1, 0, workers, w_corr,
                             a_ready)) < 0)
    return r;
  launches += r;
  if ((r = launch_finish_sc(s, u, u, Xdata, K, d.J, 1, 0, cu)) < 0) return r;
  if (emit) { pl->fresh_u = u.base; pl->fresh_v = v_fresh; pl->fresh_K = K; }
  return launches + r;
}

int umma_forward(UmmaPlan* pl, cudaStream_t s, const void* W, const __nv_bfloat16* w_shadow, const void* X,
                 const sfb_aux* aux, RowMap u, RowMap v, int* dev_status, int workers, bool for_apply) {
  const sfb_desc& d = pl->d;
  const int K = (workers > 0 ? workers : d.P) * d.B;
  int launches = 0, r;
  pl->fresh_u = pl->fresh_v = nullptr;
  pl->fresh_K = 0;
  // compensated path, apply of these very rows to follow: the kernels that write u and v also write the apply's
  // correction operands
  const bool emit = pl->x3 && for_apply && workers == 0;
  const CorrOut cu = emit ? apply_corr(pl, pl->uc, pl->ldcu, true) : CorrOut();
  CorrOut cv = emit ? apply_corr(pl, pl->vc, pl->ldcv, false) : CorrOut();
  RowMap x_rows;
  x_rows.base = const_cast<char*>(reinterpret_cast<const char*>(X));
  x_rows.ld = d.D; x_rows.B = d.B; x_rows.es = pl->es;
  x_rows.worker_stride = (long long)d.B * d.D * pl->es;
  if (d.model == SFB_MLR) {
    const bool bf16 = d.path == SFB_PATH_BF16;
    bool forked = false;
    if (v.base != nullptr && pl->side_ok) {   // v = x on the side stream, joined before this call returns its work
      if (cudaEventRecord(pl->fork, s) != cudaSuccess || cudaStreamWaitEvent(pl->side, pl->fork, 0) != cudaSuccess)
        return SFB_ERR_CUDA;
      forked = true;
    }
    // Once forked, every exit (errors included) makes `s` wait for the side stream, so the caller's stream
    // never runs ahead of the copy and a stream capture in progress stays well formed.
    auto join_side = [&]() -> int {
      if (!forked) return 0;
      if (cudaEventRecord(pl->join, pl->side) != cudaSuccess || cudaStreamWaitEvent(s, pl->join, 0) != cudaSuccess)
        return SFB_ERR_CUDA;
      return 0;
    };
    auto body = [&]() -> int {
      if (forked) {
        if ((r = launch_copy_rows(pl->side, x_rows, v, K, d.D, cv)) < 0) return r;
        launches += r;
      }
      // the GEMM epilogue leaves exp(z - local max) in u and (max, sum) per half tile; the finishing
      // pass rescales to the softmax and subtracts the one-hot label, in place
      if (pl->part_ws != nullptr) {
        // few tiles: split reduction into the partial buffers, then the plain softmax pass sums them
        RowMap pz;
        pz.base = reinterpret_cast<char*>(pl->part_ws); pz.ld = pl->ldp; pz.B = d.B; pz.es = 4;
        pz.worker_stride = (long long)d.B * pl->ldp * 4;
        const long long sstride = (long long)d.P * d.B * pl->ldp * 4;
        int ks = 1;
        if ((r = umma_forward_rows(pl, s, bf16 ? (const void*)w_shadow : W, x_rows, pz, dev_status, nullptr, nullptr,
                                   nullptr, &ks, pl->max_splits, sstride, workers, pl->x3 ? w_shadow : nullptr)) < 0)
          return r;
        launches += r;
        if ((r = launch_finish_mlr(s, pz, u, aux->labels, K, d.J, dev_status, ks, sstride, reinterpret_cast<float*>(aux->dual),
                                   aux->sdca_step, cu)) < 0)
          return r;
        launches += r;
        if (emit) { pl->fresh_u = u.base; pl->fresh_K = K; }
      } else {
        int n_parts = 0, part_cols = 0;
        if ((r = umma_forward_rows(pl, s, bf16 ? (const void*)w_shadow : W, x_rows, u, dev_status, pl->stats, &n_parts,
                                   &part_cols, nullptr, 1, 0, workers, pl->x3 ? w_shadow : nullptr)) < 0)
          return r;
        launches += r;
        if ((r = launch_finish_mlr_fused(s, u, pl->stats, n_parts, part_cols, aux->labels, K, d.J, dev_status,
                                         reinterpret_cast<float*>(aux->dual), aux->sdca_step)) < 0)
          return r;
        launches += r;
      }
      if (!forked && v.base != nullptr) {
        if ((r = launch_copy_rows(s, x_rows, v, K, d.D, cv)) < 0) return r;
        launches += r;
      }
      return 0;
    };
    const int rb = body();
    const int rj = join_side();
    if (rb < 0 || rj < 0) pl->fresh_u = nullptr;
    if (rb < 0) return rb;
    if (rj < 0) return rj;
    if (pl->fresh_u != nullptr && v.base != nullptr) pl->fresh_v = v.base;
    return launches;
  }
  // DML (TF32): the pair differences are the factor v and the GEMM operand
  if (v.base == nullptr) return SFB_ERR_ARG;
  if (pl->x3) {   // ... and the forward's own correction operand of the differences
    cv.km = reinterpret_cast<char*>(pl->xc);
    cv.atoms = (d.D + 31) / 32;
  }
  if ((r = launch_diff_rows(s, reinterpret_cast<const float*>(X), reinterpret_cast<const float*>(aux->Xb), v, K, d.D, cv)) < 0)
    return r;
  launches += r;
  if (pl->part_ws != nullptr) {
    RowMap pz;
    pz.base = reinterpret_cast<char*>(pl->part_ws); pz.ld = pl->ldp; pz.B = d.B; pz.es = 4;
    pz.worker_stride = (long long)d.B * pl->ldp * 4;
    const long long sstride = (long long)d.P * d.B * pl->ldp * 4;
    int ks = 1;
    if ((r = umma_forward_rows(pl, s, W, v, pz, dev_status, nullptr, nullptr, nullptr, &ks, pl->max_splits, sstride, workers,
                               pl->x3 ? w_shadow : nullptr, pl->x3)) < 0)
      return r;
    launches += r;
    if ((r = launch_finish_dml(s, pz, u, aux->similar, d.margin, K, d.J, ks, sstride, nullptr, cu)) < 0) return r;
    if (emit) { pl->fresh_u = u.base; pl->fresh_v = v.base; pl->fresh_K = K; }
    return launches + r;
  }
  if ((r = umma_forward_rows(pl, s, W, v, u, dev_status, nullptr, nullptr, nullptr, nullptr, 1, 0, workers,
                             pl->x3 ? w_shadow : nullptr, pl->x3)) < 0)
    return r;
  launches += r;
  if ((r = launch_finish_dml(s, u, u, aux->similar, d.margin, K, d.J, 1, 0, nullptr, cu)) < 0) return r;
  if (emit) { pl->fresh_u = u.base; pl->fresh_v = v.base; pl->fresh_K = K; }
  return launches + r;
}

// blk0: first reduction block of these rows inside the plan's correction operands; have_u / have_v: the factor stage
// already wrote them there
static int umma_apply_range(UmmaPlan* pl, cudaStream_t s, void* W, __nv_bfloat16* w_shadow, RowMap u_rows, RowMap v_rows,
                            float eta, int K, const int* dev_status, const void* directory, long long blk0, bool have_u,
                            bool have_v);

void umma_drop_corr(UmmaPlan* pl) {
  pl->fresh_u = pl->fresh_v = nullptr;
  pl->fresh_K = 0;
}

int umma_apply(UmmaPlan* pl, cudaStream_t s, void* W, __nv_bfloat16* w_shadow, RowMap u_rows, RowMap v_rows, float eta,
               int K, const int* dev_status, const void* directory) {
  const sfb_desc& d = pl->d;
  // correction operands left by the factor stage of the same step, for exactly these rows (one use)
  const bool chunked = pl->x3 && K > X3_PAIRS_PER_APPLY && K > d.B;
  const bool usable = pl->x3 && directory == nullptr && pl->fresh_K == K && (!chunked || d.B >= 32);
  const bool have_u = usable && pl->fresh_u == u_rows.base, have_v = usable && pl->fresh_v == v_rows.base;
  pl->fresh_u = pl->fresh_v = nullptr;
  pl->fresh_K = 0;
  if (chunked) {
    // The accumulator of a tile rounds toward zero once per 8 pairs (about 1.6e-8 of the sum each time), so an update
    // of very many pairs goes to W in several launches of whole worker streams, each added to W in fp32 by the
    // epilogue: more traffic on W, an error that stops growing with K.
    const int workers = K / d.B;
    int per = X3_PAIRS_PER_APPLY / d.B;
    if (per < 1) per = 1;
    int launches = 0;
    for (int w0 = 0; w0 < workers; w0 += per) {
      const int n = (workers - w0 < per) ? workers - w0 : per;
      RowMap u = u_rows, v = v_rows;
      u.base += (long long)w0 * u.worker_stride;
      v.base += (long long)w0 * v.worker_stride;
      const void* dir = directory != nullptr ? reinterpret_cast<const char*>(directory) + (size_t)w0 * 32 : nullptr;
      const long long blk0 = d.B >= 32 ? (long long)w0 * ((d.B + 31) / 32) : 0;
      const int r = umma_apply_range(pl, s, W, w_shadow, u, v, eta, n * d.B, dev_status, dir, blk0, have_u, have_v);
      if (r < 0) return r;
      launches += r;
    }
    return launches;
  }
  return umma_apply_range(pl, s, W, w_shadow, u_rows, v_rows, eta, K, dev_status, directory, 0, have_u, have_v);
}

static int umma_apply_range(UmmaPlan* pl, cudaStream_t s, void* W, __nv_bfloat16* w_shadow, RowMap u_rows, RowMap v_rows,
                            float eta, int K, const int* dev_status, const void* directory, long long blk0, bool have_u,
                            bool have_v) {
  const sfb_desc& d = pl->d;
  const int es = pl->es, CH = 128 / es;
  const int workers = K / d.B;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.B = d.B; p.P = workers;
  const int m_units = (d.J + BM - 1) / BM;
  // Folding walks the output indices (J for u, D for v) in 128-byte chunks.  D must be whole chunks.  J need not
  // be: the last chunk of a u row then also carries the first bytes of what follows the row inside the worker
  // stream (the next row, or the stream's V block: always inside the buffer), which only feeds accumulator rows
  // j >= J, and those are never written.  (The V block of the last stream ends the buffer, hence no such
  // licence for D.)
  const Variant v = pick_variant(pl, m_units, d.D, (d.D % CH) == 0, pl->x3 ? (K + 31) / 32 : 0);
  const int BK = CH * v.ka;
  if (d.B >= BK) { p.k_bb = BK; p.k_wp = 1; p.k_bpw = (d.B + BK - 1) / BK; p.k_blocks = workers * p.k_bpw; }
  else { p.k_bb = pow2_at_least(d.B); p.k_wp = BK / p.k_bb; p.k_bpw = 1; p.k_blocks = (workers + p.k_wp - 1) / p.k_wp; }
  p.m_tiles = (m_units + v.cg - 1) / v.cg;
  p.n_tiles = (d.D + v.bn - 1) / v.bn;
  p.k_splits = 1; p.k_per_split = p.k_blocks;
  // pair counts from the directory: whole reduction blocks behind a worker's last pair are left out
  p.dir = (directory != nullptr && d.B >= BK && workers <= MAX_DIR_WORKERS) ? reinterpret_cast<const uint32_t*>(directory)
                                                                            : nullptr;
  p.Mvalid = d.J; p.Nvalid = d.D;
  p.m_fastest = (d.D > d.J) ? 1 : 0;   // U is K x J, V is K x D: share the slab of the larger factor matrix
  p.a_policy = p.m_fastest ? 2 : 0;
  p.b_policy = p.m_fastest ? 0 : 2;
  p.group = APPLY_GROUP;
  p.W = reinterpret_cast<float*>(W);
  p.shadow = (d.path == SFB_PATH_BF16 || pl->x3) ? w_shadow : nullptr;
  p.w_atoms = (d.D + 31) / 32;
  p.ldw = d.D;
  p.eta = eta;
  p.status_ro = dev_status;
  p.status = const_cast<int*>(dev_status);
  p.lose_signal = pl->lose_signal;
  pl->lose_signal = 0;
  CUtensorMap tu, tv;
  // only the first `workers` streams are visible to the maps, so zero fill covers a ragged last block
  if (!encode_rows_map(&tu, es, u_rows.base, d.J, d.B, workers, (long long)u_rows.ld * es, u_rows.worker_stride, p.k_bb,
                       p.k_wp, v.fold, BM / CH, es == 4))
    return SFB_ERR_CUDA;
  if (!encode_rows_map(&tv, es, v_rows.base, d.D, d.B, workers, (long long)v_rows.ld * es, v_rows.worker_stride, p.k_bb,
                       p.k_wp, v.fold, (v.bn / v.cg) / CH, es == 4))
    return SFB_ERR_CUDA;
  // fp32 W as a 2-D map with 32 x 32 boxes (128-byte swizzle) for the epilogue's TMA stores
  CUtensorMap tw;
  {
    cuuint64_t dims[2] = {(cuuint64_t)d.D, (cuuint64_t)d.J};
    cuuint64_t strides[1] = {(cuuint64_t)d.D * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    if (get_encode()(&tw, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, W, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SFB_ERR_CUDA;
  }
  CUtensorMap tuc = tu, tvc = tv;
  int launches = 0;
  if (pl->x3) {
    // correction operands of this launch's factor rows, block by block as the kernel takes them (BK = 32 pairs)
    char* uc = reinterpret_cast<char*>(pl->uc) + blk0 * 64 * pl->ldcu * 2;
    char* vc = reinterpret_cast<char*>(pl->vc) + blk0 * 64 * pl->ldcv * 2;
    int r;
    if (!have_u) {
      if ((r = launch_split_mn(s, u_rows, d.J, workers, p.k_bb, p.k_wp, p.k_bpw, p.k_blocks, uc, pl->ldcu, true)) < 0) return r;
      launches += r;
    }
    if (!have_v) {
      if ((r = launch_split_mn(s, v_rows, d.D, workers, p.k_bb, p.k_wp, p.k_bpw, p.k_blocks, vc, pl->ldcv, false)) < 0) return r;
      launches += r;
    }
    if (!encode_corr_mn_map(&tuc, uc, pl->ldcu, (long long)p.k_blocks * 64, BM / 64) ||
        !encode_corr_mn_map(&tvc, vc, pl->ldcv, (long long)p.k_blocks * 64, (v.bn / v.cg) / 64))
      return SFB_ERR_CUDA;
  }
  const int r = dispatch_gemm<true, 0>(s, es, v, tu, tv, tw, tuc, tvc, p, pl->num_sms);
  return r < 0 ? r : launches + r;
}

}  // namespace sfb
