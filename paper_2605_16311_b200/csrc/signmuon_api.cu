// Host side of the SignMuon C ABI: validation, memory layout, tile scheduling and the
// launch sequence of one optimizer step.  See include/signmuon.h for the contract.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>
#include <queue>
#include <vector>

#include "../../include/signmuon.h"
#include "common.cuh"
#include "elementwise.cuh"
#include "ns_gemm_simt.cuh"
#include "power_iter.cuh"
#include "ns_gemm_sm100.cuh"
#include "ns_chain_sm100.cuh"

using namespace signmuon;

namespace {

constexpr size_t ALIGN = 256;
constexpr int MAX_CTAS = 1024;
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct ParamPlan {
  int64_t rows, cols, d;
  int32_t kind, wdtype, gdtype;
  int64_t s, l;
  bool wide;             // rows <= cols: Gram matrix is Y Y^T (rows x rows)
  int32_t ldy, ldq;
  uint32_t n_words, word_off;
  uint32_t chunks_per_worker;
  bool gs;               // the Newton-Schulz iteration runs in Gram space: on chip (ns_chain_kernel) for a short side up
                         // to 256, or ...
  bool gs_mem;           // ... as a chain of symmetric s x s products through memory (grouped GEMM launches) for larger
                         // matrices that are long enough for it to need fewer tensor-core operations
  // Gram-space chain through memory: Q_1 (second buffer of the Q_k ping-pong; the first is q_off / qlo_off), R_k (hi
  // only) and H_k (ping-pong); bytes into the workspace
  size_t gc_q1_off, gc_q1lo_off, gc_r_off, gc_h_off[2], gc_hlo_off[2];
  bool fused_pack;       // sign+pack happens in the last apply epilogue
  size_t mom_off;        // bytes into the state buffer
  size_t y_off[2], lo_off[2], q_off, qlo_off, scales_off, partials_off;   // bytes into the workspace (matrix params)
                         // lo_off[0] == lo_off[1] (updated in place) unless the products run in split precision
  int tmap_base;         // first of this parameter's TM_PER_PARAM tensor maps
  size_t stage_w_off, stage_g_off;                    // bytes into the host-staging buffer
  size_t pi_v_off, pi_u_off, pi_scal_off;             // power iteration (scale = spectral), bytes into the workspace
  size_t pi_start_off;                                // floats into the caller's start-vector array
  size_t s8_off;                                      // FP8 copy of the vote matrix (local polar step), bytes into the workspace
  int32_t ld8;                                        // its row pitch in bytes (cols rounded up to 16)
  bool lp_fp8;                                        // the local polar step's first Gram product runs on FP8 operands
};

// indices of a parameter's tensor maps relative to tmap_base
enum { TM_Y0_K128 = 0, TM_Y0_KBN, TM_Y0_MN, TM_Y1_K128, TM_Y1_KBN, TM_Y1_MN, TM_Q_K128, TM_Q_KBN, TM_LO0_K128, TM_MOM_F32,
       TM_Q_BOX64, TM_LO1_K128, TM_LO0_MN, TM_LO1_MN, TM_QLO_K128, TM_QLO_KBN, TM_S8,
       // Gram-space chain through memory (s x s matrices, {64 x 128} boxes: operand, C and output maps alike)
       TM_GC_Q1, TM_GC_Q1LO, TM_GC_R, TM_GC_H0, TM_GC_H0LO, TM_GC_H1, TM_GC_H1LO, TM_PER_PARAM };

struct LaunchPlan {        // one grouped GEMM launch
  size_t problem_base;     // index of its first problem in the problem array
  size_t problem_count;
  int tile_table;          // which tile table (TT_*): launches with the same problem structure share one
  bool gram;               // Gram launch (else apply launch)
};

// Tile tables.  The workers' first Gram launch and last apply launch also carry the parameters whose iteration runs in
// Gram space (they take part in no other launch), so those two launches have tables of their own.
enum { TT_GRAM_FIRST = 0, TT_APPLY_LAST, TT_GRAM, TT_APPLY, TT_LP_GRAM_FIRST, TT_LP_APPLY_LAST, TT_LP_GRAM, TT_LP_APPLY,
       TT_GC_R, TT_GC_Q, TT_GC_HR, TT_GC_F,      // launches of the Gram-space chain through memory: workers ...
       TT_LP_GC_R, TT_LP_GC_Q, TT_LP_GC_HR, TT_LP_GC_F,   // ... and local polar step (same order)
       TT_COUNT };

struct TileTable {
  std::vector<TileEntry> tiles;         // ordered by CTA
  std::vector<uint32_t> cta_start;      // [grid + 1]
  int grid = 0;            // number of tile lists = CTAs (one-CTA kernel) or CTA pairs
  int bm = 128, bn = 128;  // tile shape
  int ctas = 1;            // CTAs that share a tile
  bool long_k = false;     // tile-weighted mean contraction length >= 1536 (chooses the apply kernel's rings)
  size_t tiles_off = 0, cta_off = 0;    // bytes into the workspace
  size_t problem_base = 0, problem_count = 0;   // the launch that defines the table (others using it have the same structure)
  bool used = false;
  double flops = 0;                     // flops its tiles issue per launch
};

}  // namespace

struct signmuon_ctx {
  signmuon_config cfg;
  std::vector<signmuon_param> params;
  std::vector<ParamPlan> plan;
  std::vector<int32_t> matrix_list, plain_list, packfb_list, vote_list;
  std::vector<uint32_t> mom_starts, plain_starts, upd_starts, packfb_starts, xv_starts, xtu_starts;
  uint32_t upd_blocks = 0;
  uint32_t mom_blocks = 0, plain_blocks = 0, vote_blocks = 0, packfb_blocks = 0, xv_blocks = 0, xtu_blocks = 0;
  size_t power_start_floats = 0;          // length of the start-vector array (scale = spectral)
  const float* d_power_start = nullptr;   // caller's start vectors (device)
  int M_all = 1;                          // workers that vote (config.num_workers)
  int Lw = 1;                             // workers this context computes (momentum, Newton-Schulz, pack)
  int w_off = 0;                          // global index of its first worker
  int Wm = 1;                             // Newton-Schulz batch slots of a matrix parameter's workers: Lw, or 1 under the
                                          // Muon rule (one momentum of the mean gradient)
  bool muon = false;                      // update_rule == SIGNMUON_RULE_MUON
  bool lp = false;                        // local polar step in effect (never under the Muon rule)
  bool sharded = false;                   // Lw < M_all: the payload rows of the other workers come from elsewhere
  uint64_t words_per_worker = 0;          // payload words of one worker (the bytes it would transmit / 4)
  uint64_t bits_pitch = 0;                // words between two workers' payloads in the workspace (128-byte rows)
  int64_t entries = 0;
  size_t state_bytes = 0, workspace_bytes = 0, staging_bytes = 0;
  // workspace offsets
  size_t paramdev_stride = 0;             // bytes between two copies of the parameter table
  size_t off_status = 0, off_paramdev = 0, off_lists = 0, off_bits = 0, off_vote = 0, off_tmaps = 0,
         off_problems = 0, off_tables_end = 0;
  size_t off_list_vote = 0, off_starts_upd = 0, off_flags = 0;
  size_t off_list_matrix = 0, off_list_plain = 0, off_list_packfb = 0, off_starts_mom = 0, off_starts_plain = 0,
         off_starts_packfb = 0, off_starts_xv = 0, off_starts_xtu = 0, off_agree = 0;
  // GEMM plans
  std::vector<GemmProblem> problems;      // pointers filled at bind
  std::vector<LaunchPlan> ns_launches, lp_launches;
  TileTable tables[TT_COUNT];
  // Newton-Schulz in Gram space (short side <= 256): one chain launch between the first Gram and the last apply launch
  // Gram-space chain launches: [0] the workers' iterations, [1] the local polar step's (one problem per parameter)
  struct ChainSet {
    std::vector<ChainProblem> problems;       // pointers as workspace offsets until bind
    size_t off_problems = 0, off_order = 0, off_start = 0;
    int pairs = 0;
  } chain[2];
  int num_tmaps = 0;
  // binding
  bool split = false;      // Newton-Schulz products of the workers in split precision (scale = spectral)
  bool bound = false;
  uint8_t* d_state = nullptr;
  uint8_t* d_ws = nullptr;
  uint8_t* d_staging = nullptr;
  size_t stage_g_base = 0, stage_g_set_bytes = 0;
  // signmuon_step_host: gradients are copied on an internal stream, one step ahead of the compute
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_loaded[2] = {nullptr, nullptr}, ev_consumed[2] = {nullptr, nullptr};
  cudaEvent_t ev_weights_up = nullptr;       // the last call's weight upload has left the host-to-device copy engine
  uint64_t host_steps = 0;
  int num_sms = 0;
  // Parameter tables.  The device keeps PARAM_TABLES copies of the ParamDev table, one per set of caller
  // pointers (weights, gradients) seen recently: a caller that alternates between a few sets of buffers (two
  // gradient buffers, the two staging sets of signmuon_step_host) finds its table already on the device and
  // the step uploads nothing.  A new set takes the least recently used slot; its image is written into that
  // slot's pinned host mirror and copied asynchronously (the slot's event guards the mirror's reuse).
  std::vector<ParamDev> paramdev;         // template: everything except W and G
  ParamDev* h_tables = nullptr;           // pinned host mirrors, [PARAM_TABLES][num_params]
  cudaEvent_t ev_table[4] = {nullptr, nullptr, nullptr, nullptr};
  std::vector<const void*> table_key[4];  // W pointers then G pointers of the set a slot holds (empty: free)
  uint64_t table_used[4] = {0, 0, 0, 0};
  uint64_t table_clock = 0;
  int cur_table = 0;                      // slot of the step being enqueued
  uint64_t wait_limit_ns = DEFAULT_WAIT_LIMIT_NS;
  // fused exchange: payload words are also stored into the peers' payload buffers; flags tell when they are complete
  PeerList peers = {};                    // byte distance of every peer's payload buffer from this one
  FlagList peer_flags = {};               // every peer's flag array
  int my_rank = 0, n_ranks = 1;
  uint32_t exchange_seq = 0;              // sequence number of the last published payload
  VoteRanges vote_ranges = {};            // word ranges of the payload the vote kernel covers
  double executed_flops = 0;              // flops the scheduled tiles issue per step (known once the tile tables exist)
  int sticky = SIGNMUON_OK;
};

namespace { constexpr int PARAM_TABLES = 4; }

namespace {

bool valid_dtype(int32_t t) { return t == SIGNMUON_F32 || t == SIGNMUON_BF16; }
size_t dtype_size(int32_t t) { return t == SIGNMUON_F32 ? 4 : 2; }

// ------------------------------------------------------------------ tile scheduling (host)
// Longest-processing-time-first assignment of tiles to `grid` persistent CTAs; cost = K blocks
// of the main loop plus a constant for the epilogue.
void build_tile_table(TileTable& tt, const std::vector<GemmProblem>& probs, size_t pbase, size_t pcount,
                      int grid_limit) {
  const int bm = tt.bm, bn = tt.bn;
  struct T { TileEntry e; int cost; };
  std::vector<T> all;
  for (size_t i = 0; i < pcount; ++i) {
    const GemmProblem& pr = probs[pbase + i];
    const int tm = (pr.M + bm - 1) / bm, tn = (pr.N + bn - 1) / bn;
    // Cost in units of one K block of the main loop (about 512 cycles on a CTA pair).  Main loop and epilogue of
    // consecutive tiles overlap, so a tile costs the longer of the two; a 64-column chunk of an apply epilogue
    // (C in, combine, hi/lo out) takes about five such units, a chunk of a Gram epilogue about one (measured
    // per-chunk cycle counts).
    const int kelem = pr.fp8 ? 2 * GEMM_BK : GEMM_BK;        // elements of K per 128-byte stage row
    const int nk = ((pr.K + kelem - 1) / kelem) * (pr.nseg > 1 ? pr.nseg : 1);
    const int per_chunk = (pr.epi == EPI_GRAM) ? 1 : 5;
    for (int a = 0; a < tm; ++a)
      for (int b = (pr.sym ? a : 0); b < tn; ++b) {   // symmetric results: tiles on or above the diagonal
        const int cols = std::min(bn, pr.N - b * bn);
        const int cost = std::max(nk, per_chunk * ((cols + 63) / 64)) + 2;
        all.push_back({{(uint32_t)i, (uint16_t)a, (uint16_t)b}, cost});
      }
  }
  tt.grid = (int)std::min<size_t>((size_t)grid_limit, std::max<size_t>(all.size(), 1));
  std::stable_sort(all.begin(), all.end(), [](const T& x, const T& y) { return x.cost > y.cost; });
  std::vector<std::vector<TileEntry>> per(tt.grid);
  typedef std::pair<long long, int> Load;   // (load, cta)
  std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
  for (int c = 0; c < tt.grid; ++c) heap.push({0, c});
  for (const T& t : all) {
    Load top = heap.top();
    heap.pop();
    per[top.second].push_back(t.e);
    heap.push({top.first + t.cost, top.second});
  }
  long long ksum = 0;
  for (const T& t : all) ksum += probs[pbase + t.e.problem].K;
  tt.long_k = !all.empty() && ksum / (long long)all.size() >= 1536;
  tt.tiles.clear();
  tt.cta_start.assign(tt.grid + 1, 0);
  for (int c = 0; c < tt.grid; ++c) {
    tt.cta_start[c] = (uint32_t)tt.tiles.size();
    tt.tiles.insert(tt.tiles.end(), per[c].begin(), per[c].end());
  }
  tt.cta_start[tt.grid] = (uint32_t)tt.tiles.size();
}

size_t count_tiles(const std::vector<GemmProblem>& probs, size_t pbase, size_t pcount, int bm, int bn) {
  size_t n = 0;
  for (size_t i = 0; i < pcount; ++i) {
    const GemmProblem& pr = probs[pbase + i];
    n += (size_t)((pr.M + bm - 1) / bm) * ((pr.N + bn - 1) / bn);
  }
  return n;
}

// ------------------------------------------------------------------ GEMM problem construction
// Builds the problem list of the Gram (`gram` = true) or apply product of Newton-Schulz
// iteration k for `workers` batch slots.  Device pointers are left as byte offsets into the
// workspace (resolved at bind) in the pointer fields.
// A parameter whose iteration runs in Gram space takes part in the first Gram launch only (A_0 = Y_0 Y_0^T, stored as
// the hi/lo pair of -A_0/2 for the chain kernel) and in the last apply launch only (Y_K = T_K Y_0 with
// T_K = (3/2)^K I + F_K: product F_K Y_0 in split precision, own term (3/2)^K Mom from the float32 momentum).
void append_problems(signmuon_ctx* c, std::vector<GemmProblem>& out, bool gram, int k, int K, int workers,
                     bool local_polar_phase) {
  const bool keep = (c->cfg.flags & SIGNMUON_FLAG_KEEP_POLAR) != 0;
  for (int32_t p : c->matrix_list) {
    const ParamPlan& pl = c->plan[p];
    const bool gs = pl.gs;
    if (gs && (gram ? k != 0 : k != K - 1)) continue;
    const bool first = gs || k == 0;                 // reads the momentum (scale from memory, float32 own term)
    const int src = gs ? 0 : (k & 1), dst = gs ? 1 : ((k + 1) & 1);
    for (int w = 0; w < workers; ++w) {
      // the local polar step works in its own slot (index M) so the workers' results stay readable
      const int m = local_polar_phase ? c->Wm : w;
      GemmProblem pr;
      std::memset(&pr, 0, sizeof(pr));
      const size_t ybytes = (size_t)pl.rows * pl.ldy * 2, qbytes = (size_t)pl.s * pl.ldq * 2;
      const size_t ysrc = pl.y_off[src] + m * ybytes, ydst = pl.y_off[dst] + m * ybytes;
      const size_t q = pl.q_off + m * qbytes;
      pr.batch = m;
      pr.param = p;
      const int ty = src ? TM_Y1_K128 : TM_Y0_K128;   // first map of the source buffer
      if (gram) {
        pr.M = pr.N = (int32_t)pl.s;
        pr.K = (int32_t)pl.l;
        pr.A = pr.B = reinterpret_cast<const bf16*>(ysrc);
        if (pl.wide) {
          pr.a_sm = pr.b_sn = pl.ldy; pr.a_sk = pr.b_sk = 1;
          pr.tmapA = pl.tmap_base + ty; pr.tmapB = pl.tmap_base + ty + 1;
        } else {
          pr.a_sm = pr.b_sn = 1; pr.a_sk = pr.b_sk = pl.ldy; pr.a_mn = pr.b_mn = 1;
          pr.tmapA = pr.tmapB = pl.tmap_base + ty + 2;
        }
        pr.epi = EPI_GRAM;
        pr.out = reinterpret_cast<void*>(q);
        pr.ld_out = pl.ldq;
        pr.tma_out = 1; pr.tmapO0 = pl.tmap_base + TM_Q_K128; pr.batch_o = m;
        pr.sym = (c->cfg.flags & SIGNMUON_FLAG_SIMT_GEMM) ? 0 : 1;   // square tiles only (bm == bn in every shape)
        pr.tmapOT = pl.tmap_base + TM_Q_BOX64;
        pr.diag_share = 1;                          // A and B are the same rows of the same matrix on diagonal tiles
        if (gs && pl.gs_mem) {
          // -A/2 as a hi/lo pair for the chain through memory: one segment (the contraction is long enough for the
          // operands' rounding to average out), upper tiles only, hi part mirrored for the chain's operand loads
          pr.gram_lo = 1;
          pr.mirror_hi = 1;
          pr.out_lo = reinterpret_cast<bf16*>(pl.qlo_off + m * qbytes);
          pr.tmapO1 = pl.tmap_base + TM_QLO_K128;
        } else if (local_polar_phase && gs) {       // -A/2 as a hi/lo pair for the chain; the +-1 operands are exact
          pr.gram_lo = 1;
          pr.sym = 0;
          pr.out_lo = reinterpret_cast<bf16*>(pl.qlo_off + m * qbytes);
          pr.tmapO1 = pl.tmap_base + TM_QLO_K128;
        } else if ((c->split && !local_polar_phase) || gs) {   // -A/2 as a hi/lo pair, both triangles computed
          pr.gram_lo = 1;
          pr.sym = 0;
          pr.diag_share = 0;                        // the segments pair different operands
          pr.out_lo = reinterpret_cast<bf16*>(pl.qlo_off + m * qbytes);
          pr.tmapO1 = pl.tmap_base + TM_QLO_K128;
          // Y Y^T ~ Yhi Yhi^T + Yhi Ylo^T + Ylo Yhi^T: the off-diagonal entries of the Gram matrix are small sums of
          // products, and dropping the lo part would leave them with the operands' 2^-9 relative rounding
          pr.nseg = 3;
          const int lk = src ? TM_LO1_K128 : TM_LO0_K128, lmn = src ? TM_LO1_MN : TM_LO0_MN;
          if (pl.wide) {
            pr.tmapA2 = pr.tmapA;             pr.tmapB2 = pl.tmap_base + lk;     // (a K-major box of 128 rows serves as B)
            pr.tmapA3 = pl.tmap_base + lk;    pr.tmapB3 = pr.tmapB;
          } else {
            pr.tmapA2 = pr.tmapA;             pr.tmapB2 = pl.tmap_base + lmn;
            pr.tmapA3 = pl.tmap_base + lmn;   pr.tmapB3 = pr.tmapB;
          }
        }
        if (k == 0 && local_polar_phase && pl.lp_fp8) {
          // S S^T of the exact +-1 vote matrix: E4M3 operands (one byte per entry, twice the tensor-core rate);
          // products are +-1 and their fp32 sums are exact integers, so the result equals the bf16 product's bit for bit
          pr.fp8 = 1;
          pr.A = pr.B = reinterpret_cast<const bf16*>(pl.s8_off);
          pr.tmapA = pr.tmapB = pl.tmap_base + TM_S8;
          pr.batch = 0;                              // the FP8 copy has a single slot
        }
        if (first) {
          if (local_polar_phase) pr.scale_imm = (float)(1.0 / ((double)pl.rows * (double)pl.cols));
          else pr.scale_ptr = reinterpret_cast<const float*>(pl.scales_off + (size_t)m * 8);
        } else {
          pr.scale_imm = 1.f;
        }
      } else {
        pr.M = (int32_t)pl.rows; pr.N = (int32_t)pl.cols; pr.K = (int32_t)pl.s;
        // the s x s factor: -A_k/2 of this iteration, or F_K when the iteration ran in Gram space (left in the Gram
        // buffers by the on-chip chain, in the H buffer of parity K by the chain through memory)
        size_t qf = q;
        int tq = TM_Q_K128, tq_b = TM_Q_KBN;
        if (gs && pl.gs_mem) {
          qf = pl.gc_h_off[K & 1] + m * qbytes;
          tq = tq_b = (K & 1) ? TM_GC_H1 : TM_GC_H0;
        }
        if (pl.wide) {                      // Y' = (3/2 I - A/2) Y : A operand Q, B operand Y (contiguous along N)
          pr.A = reinterpret_cast<const bf16*>(qf); pr.a_sm = pl.ldq; pr.a_sk = 1;
          pr.B = reinterpret_cast<const bf16*>(ysrc); pr.b_sn = 1; pr.b_sk = pl.ldy; pr.b_mn = 1;
          pr.tmapA = pl.tmap_base + tq; pr.tmapB = pl.tmap_base + ty + 2;
        } else {                            // Y' = Y (3/2 I - A/2) : A operand Y, B operand Q (symmetric)
          pr.A = reinterpret_cast<const bf16*>(ysrc); pr.a_sm = pl.ldy; pr.a_sk = 1;
          pr.B = reinterpret_cast<const bf16*>(qf); pr.b_sn = pl.ldq; pr.b_sk = 1;
          pr.tmapA = pl.tmap_base + ty; pr.tmapB = pl.tmap_base + tq_b;
        }
        const bool split = c->split && !local_polar_phase;
        const size_t lo = pl.lo_off[split ? src : 0] + m * ybytes;       // lo part of Y_k
        const size_t lo_dst = pl.lo_off[split ? dst : 0] + m * ybytes;   // lo part of Y_{k+1}
        const int tlo = split && src ? TM_LO1_K128 : TM_LO0_K128, tlo_dst = split && dst ? TM_LO1_K128 : TM_LO0_K128;
        pr.own_coef = gs ? (float)std::pow(1.5, (double)K) : 1.5f;
        if (gs && pl.gs_mem) {
          // F_K Y_0 in one segment (hi parts): over a contraction this long the operands' rounding averages out as it
          // does in every product of the iteration on the full matrix
        } else if (split || gs) {      // Q Y ~ Qhi Yhi + Qlo Yhi + Qhi Ylo (three operand segments along K)
          pr.nseg = local_polar_phase ? 2 : 3;        // (the +-1 vote matrix has no lo part)
          const int tlo_mn = src ? TM_LO1_MN : TM_LO0_MN;
          if (pl.wide) {
            pr.tmapA2 = pl.tmap_base + TM_QLO_K128; pr.tmapB2 = pr.tmapB;
            pr.tmapA3 = pr.tmapA;                   pr.tmapB3 = pl.tmap_base + tlo_mn;
          } else {
            pr.tmapA2 = pr.tmapA;                   pr.tmapB2 = pl.tmap_base + TM_QLO_KBN;
            pr.tmapA3 = pl.tmap_base + tlo;         pr.tmapB3 = pr.tmapB;
          }
        }
        if (first && !local_polar_phase) {           // own term from the float32 momentum itself
          pr.c_mode = C_F32;
          pr.C = reinterpret_cast<const void*>(pl.mom_off + (size_t)m * pl.d * 4);   // offset into the state buffer
          pr.ldc = pl.cols;
        } else {
          pr.c_mode = first ? C_BF16 : C_HILO;       // the +-1 vote matrix is exact in bf16
          pr.C = reinterpret_cast<const void*>(ysrc);
          pr.C_lo = first ? nullptr : reinterpret_cast<const bf16*>(lo);
          pr.ldc = pl.ldy;
        }
        pr.out = reinterpret_cast<void*>(ydst);
        pr.out_lo = reinterpret_cast<bf16*>(lo_dst);
        pr.ld_out = pl.ldy;
        // TMA-staged epilogue: possible whenever the row pitches are multiples of 16 bytes
        pr.tma_out = 1;
        pr.tmapO0 = pl.tmap_base + (dst ? TM_Y1_K128 : TM_Y0_K128);
        pr.tmapO1 = pl.tmap_base + tlo_dst;
        pr.batch_o = m;
        pr.batch_c = m;
        if (pr.c_mode == C_F32) {
          pr.tma_c = (pl.cols % 4 == 0) ? 1 : 0;
          pr.tmapC0 = pl.tmap_base + TM_MOM_F32;
        } else {
          pr.tma_c = 1;
          pr.tmapC0 = pl.tmap_base + ty;
          pr.tmapC1 = pl.tmap_base + tlo;
        }
        if (first) {
          if (local_polar_phase) pr.scale_imm = (float)(1.0 / std::sqrt((double)pl.rows * (double)pl.cols));
          else pr.scale_ptr = reinterpret_cast<const float*>(pl.scales_off + (size_t)m * 8 + 4);
        } else {
          pr.scale_imm = 1.f;
        }
        const bool last = (k == K - 1);
        if (gs && !last) continue;                   // (unreachable: filtered above)
        if (!last) pr.epi = EPI_APPLY;
        else if (local_polar_phase || c->muon) pr.epi = EPI_APPLY_UPDATE;   // W <- W - eta Y_K (local polar step; Muon rule)
        else if (pl.fused_pack) {
          pr.epi = EPI_APPLY_PACK;
          pr.store_out = keep ? 1 : 0;
          // payload word of this (param, worker): resolved at bind from off_bits
          pr.bits_out = reinterpret_cast<uint32_t*>((size_t)(c->w_off + m) * c->bits_pitch * 4 + (size_t)pl.word_off * 4);
        } else pr.epi = EPI_APPLY;
        // (the lo part of the source is an operand of this product's other tiles: it must not be overwritten; nothing
        // reads the lo part of Y_K)
        if (gs) pr.hi_only = 1;
      }
      out.push_back(pr);
    }
  }
}

// Problems of the Gram-space chain through memory (parameters with gs_mem), one launch stage at a time.  With
// Q_k = -A_k / 2 (Q_0 is what the first Gram launch stores) and T_k = (3/2)^k (I + H_k) the printed iteration reads
//     R_k     = Q_k Q_k + 3 Q_k
//     Q_{k+1} = Q_k R_k + 9/4 Q_k                          (= -A_{k+1} / 2 with A_{k+1} = P_k A_k P_k)
//     H_{k+1} = 2/3 (Q_k H_k + Q_k + 3/2 H_k),  H_1 = 2/3 Q_0,  F_K = (3/2)^K H_K     (T_{k+1} = P_k T_k)
// Every line is one product with the apply epilogue y = scale (acc + own C + c2 C2): the tensor-core operands are the
// hi parts, the linear terms enter as hi + lo.  All matrices are polynomials in A_0: symmetric and commuting, so only
// the tiles on or above the diagonal are computed; the hi part (the next products' operand) is also stored mirrored,
// the lo part is only ever read as a linear term of the same tile.  H_1 is never stored:
// H_2 = 4/9 (Q_1 Q_0 + 3/2 Q_0 + 3/2 Q_1) uses Q_0 directly.  The last H launch scales its result to F_K.
enum { GC_R = 0, GC_Q, GC_H };
void append_gc_problems(signmuon_ctx* c, std::vector<GemmProblem>& out, int what, int k, int K, bool local_polar_phase) {
  for (int32_t p : c->matrix_list) {
    const ParamPlan& pl = c->plan[p];
    if (!pl.gs_mem) continue;
    const size_t qbytes = (size_t)pl.s * pl.ldq * 2;
    // (the local polar step works in its own batch slot, index Wm)
    for (int m = local_polar_phase ? c->Wm : 0; m < (local_polar_phase ? c->Wm + 1 : c->Wm); ++m) {
      // Q_k lives in buffer k & 1 (buffer 0 = the Gram launch's output), H_k in H buffer k & 1
      auto q_hi = [&](int kk) { return ((kk & 1) ? pl.gc_q1_off : pl.q_off) + m * qbytes; };
      auto q_lo = [&](int kk) { return ((kk & 1) ? pl.gc_q1lo_off : pl.qlo_off) + m * qbytes; };
      auto q_map = [&](int kk, bool lo) { return pl.tmap_base + ((kk & 1) ? (lo ? TM_GC_Q1LO : TM_GC_Q1) : (lo ? TM_QLO_K128 : TM_Q_K128)); };
      auto h_map = [&](int kk, bool lo) { return pl.tmap_base + ((kk & 1) ? TM_GC_H1 : TM_GC_H0) + (lo ? 1 : 0); };
      GemmProblem pr;
      std::memset(&pr, 0, sizeof(pr));
      pr.M = pr.N = pr.K = (int32_t)pl.s;
      pr.a_sm = pr.b_sn = pl.ldq; pr.a_sk = pr.b_sk = 1;
      pr.batch = pr.batch_c = pr.batch_o = m;
      pr.param = p;
      pr.epi = EPI_APPLY;
      pr.c_mode = C_HILO;
      pr.ldc = pr.ld_out = pl.ldq;
      pr.tma_c = pr.tma_out = 1;
      pr.scale_imm = 1.f;
      pr.sym = 1;
      pr.mirror_hi = 1;
      pr.A = reinterpret_cast<const bf16*>(q_hi(k));
      pr.tmapA = q_map(k, false);
      pr.C = reinterpret_cast<const void*>(q_hi(k));
      pr.C_lo = reinterpret_cast<const bf16*>(q_lo(k));
      pr.tmapC0 = q_map(k, false); pr.tmapC1 = q_map(k, true);
      if (what == GC_R) {
        pr.B = pr.A; pr.tmapB = pr.tmapA;
        pr.own_coef = 3.f;
        pr.out = reinterpret_cast<void*>(pl.gc_r_off + m * qbytes);
        pr.out_lo = reinterpret_cast<bf16*>(pl.gc_r_off + m * qbytes);     // (never written: hi only)
        pr.hi_only = 1;
        pr.tmapO0 = pr.tmapO1 = pl.tmap_base + TM_GC_R;
      } else if (what == GC_Q) {
        pr.B = reinterpret_cast<const bf16*>(pl.gc_r_off + m * qbytes); pr.tmapB = pl.tmap_base + TM_GC_R;
        pr.own_coef = 2.25f;
        pr.out = reinterpret_cast<void*>(q_hi(k + 1));
        pr.out_lo = reinterpret_cast<bf16*>(q_lo(k + 1));
        pr.tmapO0 = q_map(k + 1, false); pr.tmapO1 = q_map(k + 1, true);
      } else {
        const bool from_q0 = (k == 1);       // H_1 = 2/3 Q_0 is not stored
        pr.C2 = reinterpret_cast<const bf16*>(q_hi(k));
        pr.C2_lo = reinterpret_cast<const bf16*>(q_lo(k));
        if (from_q0) {
          pr.B = reinterpret_cast<const bf16*>(q_hi(0)); pr.tmapB = q_map(0, false);
          pr.C = reinterpret_cast<const void*>(q_hi(0)); pr.C_lo = reinterpret_cast<const bf16*>(q_lo(0));
          pr.tmapC0 = q_map(0, false); pr.tmapC1 = q_map(0, true);
          pr.c2_coef = 1.5f;
        } else {
          pr.B = reinterpret_cast<const bf16*>(pl.gc_h_off[k & 1] + m * qbytes); pr.tmapB = h_map(k, false);
          pr.C = reinterpret_cast<const void*>(pl.gc_h_off[k & 1] + m * qbytes);
          pr.C_lo = reinterpret_cast<const bf16*>(pl.gc_hlo_off[k & 1] + m * qbytes);
          pr.tmapC0 = h_map(k, false); pr.tmapC1 = h_map(k, true);
          pr.c2_coef = 1.f;
        }
        pr.own_coef = 1.5f;
        double scale = from_q0 ? 4.0 / 9.0 : 2.0 / 3.0;
        const bool final_h = (k == K - 1);
        if (final_h) scale *= std::pow(1.5, (double)K);
        pr.scale_imm = (float)scale;
        pr.hi_only = final_h ? 1 : 0;        // F_K is an operand only
        pr.out = reinterpret_cast<void*>(pl.gc_h_off[(k + 1) & 1] + m * qbytes);
        pr.out_lo = reinterpret_cast<bf16*>(pl.gc_hlo_off[(k + 1) & 1] + m * qbytes);
        pr.tmapO0 = h_map(k + 1, false); pr.tmapO1 = h_map(k + 1, true);
      }
      out.push_back(pr);
    }
  }
}

int plan_layout(signmuon_ctx* c) {
  const int M = c->Wm;                    // batch slots of a matrix parameter: this context's own workers (1: Muon rule)
  const int K = c->cfg.ns_steps;
  size_t state = 0;
  uint64_t words = 0;
  for (size_t p = 0; p < c->params.size(); ++p) {
    const signmuon_param& sp = c->params[p];
    ParamPlan pl;
    std::memset(&pl, 0, sizeof(pl));
    pl.rows = sp.rows; pl.cols = sp.cols; pl.d = sp.rows * sp.cols;
    pl.kind = sp.kind; pl.wdtype = sp.weight_dtype; pl.gdtype = sp.grad_dtype;
    pl.s = std::min(sp.rows, sp.cols); pl.l = std::max(sp.rows, sp.cols);
    pl.wide = sp.rows <= sp.cols;
    pl.ldy = (int32_t)round_up((size_t)sp.cols, 8);
    pl.ldq = (int32_t)round_up((size_t)pl.s, 8);
    pl.n_words = (uint32_t)((pl.d + 31) / 32);
    pl.word_off = (uint32_t)words;
    words += pl.n_words;
    pl.chunks_per_worker = (uint32_t)((pl.d + MOM_CHUNK - 1) / MOM_CHUNK);
    pl.fused_pack = (sp.kind == SIGNMUON_PARAM_MATRIX) && K > 0 && (sp.cols % 32 == 0) && !c->muon;
    // Gram-space iteration for short sides up to 256: needs at least two iterations to pay, the tensor-core kernels,
    // and the Frobenius scale (with the spectral scale the products already run in split precision the regular way)
    const bool gs_ok = sp.kind == SIGNMUON_PARAM_MATRIX && K >= 2 &&
                       !(c->cfg.flags & (SIGNMUON_FLAG_SIMT_GEMM | SIGNMUON_FLAG_NO_GRAM_SPACE)) &&
                       c->cfg.ns_scale == SIGNMUON_SCALE_FRO;
    // Larger short sides: the same chain as symmetric products through memory, where it takes fewer tensor-core
    // operations.  On the tiles actually computed an iteration on the full matrix costs about 3.06 s^2 l multiply-adds
    // (Gram, upper tiles only, plus apply); the chain costs one Gram and one apply product (3.06 s^2 l) plus 3 (K - 1)
    // symmetric s^3 products (about 0.53 s^3 each on the upper tiles).
    // Measured: long sides from twice the short one gain (ResNet-50's 512 x 1024 ... 1000 x 2048, GPT-2's 768 x 2304
    // and 768 x 3072, Llama's 4096 x 11008), square matrices lose a little (768^2, 4096^2).
    pl.gs_mem = gs_ok && pl.s > 256 && 2 * pl.l >= 3 * pl.s;
    pl.gs = gs_ok && (pl.s <= 256 || pl.gs_mem);
    pl.ld8 = (int32_t)round_up((size_t)sp.cols, 16);
    pl.lp_fp8 = sp.kind == SIGNMUON_PARAM_MATRIX && c->lp && K > 0 &&
                !(c->cfg.flags & (SIGNMUON_FLAG_SIMT_GEMM | SIGNMUON_FLAG_LP_GRAM_BF16));
    pl.mom_off = state;
    state += round_up((size_t)(sp.kind == SIGNMUON_PARAM_MATRIX ? c->Wm : c->Lw) * pl.d * 4, ALIGN);
    c->plan.push_back(pl);
    if (sp.kind == SIGNMUON_PARAM_MATRIX) c->matrix_list.push_back((int32_t)p);
    else c->plain_list.push_back((int32_t)p);
    c->entries += pl.d;
  }
  // The chain through memory adds 2K - 1 launches to a step (to the workers' iterations, and again to the local polar
  // step): measured, that pays once the matrices that would take it hold about 8 M (entry, worker) pairs together
  // (512 x 2048 from 8 workers on, 1024 x 4096 from 2); below that they iterate on the full matrix.
  {
    double pairs = 0;
    for (const ParamPlan& pl : c->plan) if (pl.gs_mem) pairs += (double)pl.d * c->Wm;
    if (pairs < 8.0e6)
      for (ParamPlan& pl : c->plan) if (pl.gs_mem) pl.gs_mem = pl.gs = false;
  }
  if (words >= (1ull << 32)) return SIGNMUON_ERR_BAD_SHAPE;
  c->words_per_worker = words;
  c->bits_pitch = round_up((size_t)words, 32);
  c->state_bytes = state;

  // block ranges of the element-wise kernels
  uint64_t b = 0;
  for (int32_t p : c->matrix_list) { c->mom_starts.push_back((uint32_t)b); b += (uint64_t)M * c->plan[p].chunks_per_worker; }
  if (b >= (1ull << 31)) return SIGNMUON_ERR_BAD_SHAPE;
  c->mom_blocks = (uint32_t)b;
  b = 0;
  for (int32_t p : c->plain_list) { c->plain_starts.push_back((uint32_t)b); b += (uint64_t)((c->plan[p].d + PLAIN_CHUNK - 1) / PLAIN_CHUNK); }
  if (b >= (1ull << 31)) return SIGNMUON_ERR_BAD_SHAPE;
  c->plain_blocks = (uint32_t)b;
  b = 0;
  if (!c->muon) c->vote_list = c->matrix_list;
  if (c->sharded) {       // the plain parameters' vote also waits for the exchange: every parameter goes through the vote kernel
    c->vote_list.clear();
    for (size_t p = 0; p < c->params.size(); ++p) c->vote_list.push_back((int32_t)p);
  }
  // vote kernel: the payload words of these parameters as a few contiguous ranges with bounds rounded outwards to
  // four words (parameters follow one another in the payload, so neighbours merge); too many ranges: everything
  {
    VoteRanges vr = {};
    std::vector<std::pair<int64_t, int64_t>> rg;
    for (int32_t p : c->vote_list) {
      const ParamPlan& pl = c->plan[p];
      const int64_t lo = (int64_t)pl.word_off / 4 * 4, hi = ((int64_t)pl.word_off + pl.n_words + 3) / 4 * 4;
      if (!rg.empty() && lo <= rg.back().second) rg.back().second = std::max(rg.back().second, hi);
      else rg.push_back({lo, hi});
    }
    if ((int)rg.size() > MAX_VOTE_RANGES) rg.assign(1, {0, ((int64_t)words + 3) / 4 * 4});
    vr.n = (int32_t)rg.size();
    int64_t quads = 0;
    for (int i = 0; i < vr.n; ++i) {
      vr.begin[i] = rg[i].first;
      vr.quads_before[i] = quads;
      quads += (rg[i].second - rg[i].first) / 4;
    }
    vr.quads_before[vr.n] = quads;
    c->vote_ranges = vr;
    c->vote_blocks = (uint32_t)((quads + VOTE_THREADS - 1) / VOTE_THREADS);
  }
  // update kernel: blocks of UPD_VECS 128-bit vectors (8 bf16 or 4 float32 entries each; the +-1 matrix is bf16)
  b = 0;
  for (int32_t p : c->vote_list) {
    const ParamPlan& pl = c->plan[p];
    const bool sbar = c->lp && K > 0 && pl.kind == SIGNMUON_PARAM_MATRIX;
    const uint64_t per_block = (uint64_t)UPD_VECS * ((sbar || pl.wdtype == SIGNMUON_BF16) ? 8 : 4);
    c->upd_starts.push_back((uint32_t)b);
    b += ((uint64_t)pl.d + per_block - 1) / per_block;
  }
  if (b >= (1ull << 31)) return SIGNMUON_ERR_BAD_SHAPE;
  c->upd_blocks = (uint32_t)b;
  b = 0;
  for (int32_t p : c->matrix_list) {
    if (c->plan[p].fused_pack || c->muon) continue;     // (nothing is packed under the Muon rule)
    c->packfb_list.push_back(p);
    c->packfb_starts.push_back((uint32_t)b);
    b += (uint64_t)M * ((c->plan[p].d + PACK_CHUNK - 1) / PACK_CHUNK);
  }
  if (b >= (1ull << 31)) return SIGNMUON_ERR_BAD_SHAPE;
  c->packfb_blocks = (uint32_t)b;
  const bool spectral = c->cfg.ns_scale == SIGNMUON_SCALE_SPECTRAL && K > 0;
  // With sigma ~ ||Mom||_op the product term of the iteration is as large as the own term: the products then
  // run in split precision (not on the diagnostic CUDA-core kernel, which has no operand segments).
  c->split = spectral && !(c->cfg.flags & SIGNMUON_FLAG_SIMT_GEMM);
  if (spectral) {
    uint64_t bx = 0, bt = 0;
    size_t nf = 0;
    for (int32_t p : c->matrix_list) {
      ParamPlan& pl = c->plan[p];
      c->xv_starts.push_back((uint32_t)bx);
      c->xtu_starts.push_back((uint32_t)bt);
      bx += (uint64_t)M * ((pl.rows + PI_ROWS_PER_BLOCK - 1) / PI_ROWS_PER_BLOCK);
      bt += (uint64_t)M * ((pl.cols + PI_COLS_PER_BLOCK - 1) / PI_COLS_PER_BLOCK);
      pl.pi_start_off = nf;
      nf += (size_t)M * pl.cols;
    }
    if (bx >= (1ull << 31) || bt >= (1ull << 31)) return SIGNMUON_ERR_BAD_SHAPE;
    c->xv_blocks = (uint32_t)bx;
    c->xtu_blocks = (uint32_t)bt;
    c->power_start_floats = nf;
  }

  // workspace layout: small tables first, then the large buffers
  size_t off = 0;
  c->off_status = off; off += ALIGN;
  c->paramdev_stride = round_up(c->params.size() * sizeof(ParamDev), ALIGN);
  c->off_paramdev = off; off += PARAM_TABLES * c->paramdev_stride;
  auto place = [&](size_t& slot, size_t bytes) { slot = off; off += round_up(std::max<size_t>(bytes, 4), ALIGN); };
  place(c->off_list_matrix, c->matrix_list.size() * 4);
  place(c->off_list_plain, c->plain_list.size() * 4);
  place(c->off_list_packfb, c->packfb_list.size() * 4);
  place(c->off_list_vote, c->vote_list.size() * 4);
  place(c->off_starts_mom, c->mom_starts.size() * 4);
  place(c->off_starts_plain, c->plain_starts.size() * 4);
  place(c->off_starts_upd, c->upd_starts.size() * 4);
  place(c->off_starts_packfb, c->packfb_starts.size() * 4);
  place(c->off_agree, (size_t)c->M_all * 8);
  place(c->off_flags, 64 * 4);
  place(c->off_starts_xv, c->xv_starts.size() * 4);
  place(c->off_starts_xtu, c->xtu_starts.size() * 4);
  for (int32_t p : c->matrix_list) {
    ParamPlan& pl = c->plan[p];
    pl.scales_off = off; off += round_up((size_t)M * 8, ALIGN);
    pl.partials_off = off; off += round_up((size_t)M * pl.chunks_per_worker * 4, ALIGN);
    if (spectral) {
      pl.pi_v_off = off; off += round_up((size_t)M * pl.cols * 4, ALIGN);
      pl.pi_u_off = off; off += round_up((size_t)M * pl.rows * 4, ALIGN);
      pl.pi_scal_off = off; off += round_up((size_t)M * 8, ALIGN);
    }
  }
  c->off_bits = off; off += round_up((size_t)c->M_all * c->bits_pitch * 4, ALIGN);
  c->off_vote = off; off += round_up((size_t)c->bits_pitch * 4, ALIGN);
  // tensor maps
  c->off_tmaps = off;
  int nt = 0;
  for (int32_t p : c->matrix_list) { c->plan[p].tmap_base = nt; nt += TM_PER_PARAM; }
  c->num_tmaps = nt;
  off += round_up((size_t)std::max(nt, 1) * sizeof(CUtensorMap), ALIGN);
  // Newton-Schulz operand buffers
  for (int32_t p : c->matrix_list) {
    ParamPlan& pl = c->plan[p];
    const size_t slots = (size_t)M + (c->lp ? 1 : 0);
    const size_t ybytes = round_up(slots * pl.rows * pl.ldy * 2, 1024);
    pl.y_off[0] = off; off += ybytes;
    pl.y_off[1] = off; off += ybytes;
    pl.lo_off[0] = pl.lo_off[1] = off; off += ybytes;
    pl.q_off = off; off += round_up(slots * pl.s * pl.ldq * 2, 1024);
    if (c->split) { pl.lo_off[1] = off; off += ybytes; }
    if (c->split || pl.gs) { pl.qlo_off = off; off += round_up(slots * pl.s * pl.ldq * 2, 1024); }
    if (pl.gs_mem) {
      const size_t qb = round_up(slots * pl.s * pl.ldq * 2, 1024);
      pl.gc_q1_off = off; off += qb;
      pl.gc_q1lo_off = off; off += qb;
      pl.gc_r_off = off; off += qb;
      for (int i = 0; i < 2; ++i) { pl.gc_h_off[i] = off; off += qb; pl.gc_hlo_off[i] = off; off += qb; }
    }
    if (pl.lp_fp8) { pl.s8_off = off; off += round_up((size_t)pl.rows * pl.ld8, 1024); }
  }
  // GEMM problems: K x (gram, apply) for the workers, and again for the local polar step
  c->problems.clear();
  c->ns_launches.clear();
  c->lp_launches.clear();
  for (int t = 0; t < TT_COUNT; ++t) c->tables[t] = TileTable();
  auto add_launch = [&](std::vector<LaunchPlan>& ls, bool gram, int k, int workers, bool lp_phase, int table) {
    LaunchPlan lp;
    lp.problem_base = c->problems.size();
    append_problems(c, c->problems, gram, k, K, workers, lp_phase);
    lp.problem_count = c->problems.size() - lp.problem_base;
    lp.tile_table = table;
    lp.gram = gram;
    if (lp.problem_count == 0) return;                 // (every parameter of this launch iterates in Gram space)
    TileTable& tt = c->tables[table];
    if (!tt.used) { tt.used = true; tt.problem_base = lp.problem_base; tt.problem_count = lp.problem_count; }
    ls.push_back(lp);
  };
  // one launch of the Gram-space chain through memory: the problems of `stages` (GC_*) of iteration k
  auto add_gc_launch = [&](std::vector<LaunchPlan>& ls, std::initializer_list<int> stages, int k, bool lp_phase, int table) {
    LaunchPlan lp;
    lp.problem_base = c->problems.size();
    for (int what : stages) append_gc_problems(c, c->problems, what, k, K, lp_phase);
    lp.problem_count = c->problems.size() - lp.problem_base;
    lp.tile_table = table;
    lp.gram = false;
    if (lp.problem_count == 0) return;
    TileTable& tt = c->tables[table];
    if (!tt.used) { tt.used = true; tt.problem_base = lp.problem_base; tt.problem_count = lp.problem_count; }
    ls.push_back(lp);
  };
  // the chain through memory follows the first Gram launch (tables: R, Q, HR, F in this order from `t0`)
  auto add_gc_chain = [&](std::vector<LaunchPlan>& ls, bool lp_phase, int t0) {
    if (K < 2) return;
    add_gc_launch(ls, {GC_R}, 0, lp_phase, t0);
    add_gc_launch(ls, {GC_Q}, 0, lp_phase, t0 + 1);
    for (int kk = 1; kk <= K - 2; ++kk) {
      add_gc_launch(ls, {GC_H, GC_R}, kk, lp_phase, t0 + 2);
      add_gc_launch(ls, {GC_Q}, kk, lp_phase, t0 + 1);
    }
    add_gc_launch(ls, {GC_H}, K - 1, lp_phase, t0 + 3);
  };
  if (!c->matrix_list.empty()) {
    for (int k = 0; k < K; ++k) {
      add_launch(c->ns_launches, true, k, M, false, k == 0 ? TT_GRAM_FIRST : TT_GRAM);
      if (k == 0) add_gc_chain(c->ns_launches, false, TT_GC_R);
      add_launch(c->ns_launches, false, k, M, false, k == K - 1 ? TT_APPLY_LAST : TT_APPLY);
    }
    if (c->lp) {
      for (int k = 0; k < K; ++k) {
        add_launch(c->lp_launches, true, k, 1, true, k == 0 ? TT_LP_GRAM_FIRST : TT_LP_GRAM);
        if (k == 0) add_gc_chain(c->lp_launches, true, TT_LP_GC_R);
        add_launch(c->lp_launches, false, k, 1, true, k == K - 1 ? TT_LP_APPLY_LAST : TT_LP_APPLY);
      }
    }
  }
  c->off_problems = off; off += round_up(c->problems.size() * sizeof(GemmProblem), ALIGN);
  // tile tables (sizes do not depend on the SM count; the CTA split is made at bind)
  for (int t = 0; t < TT_COUNT; ++t) {
    TileTable& tt = c->tables[t];
    const bool pair = !(c->cfg.flags & (SIGNMUON_FLAG_GEMM_1CTA | SIGNMUON_FLAG_SIMT_GEMM));
    tt.ctas = pair ? 2 : 1;
    tt.bm = pair ? 256 : 128;
    tt.bn = pair ? 256 : 128;
    size_t ntiles = 0;
    if (tt.used) ntiles = count_tiles(c->problems, tt.problem_base, tt.problem_count, tt.bm, tt.bn);
    tt.tiles_off = off; off += round_up(std::max<size_t>(ntiles, 1) * sizeof(TileEntry), ALIGN);
    tt.cta_off = off; off += round_up((MAX_CTAS + 1) * 4, ALIGN);
  }
  // chain problems: one per (Gram-space parameter, worker), and one per parameter in the local polar step's slot;
  // -A_0/2 in, F_K out (the hi/lo Gram buffers)
  for (int set = 0; set < 2; ++set) {
    signmuon_ctx::ChainSet& cs = c->chain[set];
    cs.problems.clear();
    for (int32_t p : c->matrix_list) {
      const ParamPlan& pl = c->plan[p];
      if (!pl.gs || pl.gs_mem || (set == 1 && !c->lp)) continue;
      const size_t qbytes = (size_t)pl.s * pl.ldq * 2;
      for (int m = (set ? M : 0); m < (set ? M + 1 : M); ++m) {
        ChainProblem cp;
        cp.q_hi = reinterpret_cast<bf16*>(pl.q_off + m * qbytes);
        cp.q_lo = reinterpret_cast<bf16*>(pl.qlo_off + m * qbytes);
        cp.s = (int32_t)pl.s;
        cp.ldq = pl.ldq;
        cs.problems.push_back(cp);
      }
    }
    cs.off_problems = off; off += round_up(std::max<size_t>(cs.problems.size(), 1) * sizeof(ChainProblem), ALIGN);
    cs.off_order = off; off += round_up(std::max<size_t>(cs.problems.size(), 1) * 4, ALIGN);
    cs.off_start = off; off += round_up((MAX_CTAS + 1) * 4, ALIGN);
  }
  c->off_tables_end = off;
  c->workspace_bytes = off;

  // host staging: W of every parameter once, G of every parameter twice (two sets, so that the copy of the
  // next step's gradients can run while this step computes)
  size_t st = 0;
  for (ParamPlan& pl : c->plan) { pl.stage_w_off = st; st += round_up((size_t)pl.d * dtype_size(pl.wdtype), ALIGN); }
  c->stage_g_base = st;
  size_t gs = 0;
  for (ParamPlan& pl : c->plan) { pl.stage_g_off = gs; gs += round_up((size_t)c->Lw * pl.d * dtype_size(pl.gdtype), ALIGN); }
  c->stage_g_set_bytes = gs;
  c->staging_bytes = st + 2 * gs;
  return SIGNMUON_OK;
}

PFN_cuTensorMapEncodeTiled_v12000 get_encode_fn() {
  static std::once_flag once;
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  });
  return fn;
}

// 3-D bf16 tensor {inner, rows, batch} with a {64, box_rows, 1} box and 128-byte swizzle.
bool encode_map(CUtensorMap* map, void* base, uint64_t inner, uint64_t rows, uint64_t batch, uint64_t pitch_elems,
                uint64_t batch_elems, uint32_t box_rows, bool f32 = false) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = get_encode_fn();
  if (!fn) return false;
  const uint64_t es = f32 ? 4 : 2;
  cuuint64_t gdim[3] = {inner, rows, batch};
  cuuint64_t gstr[2] = {pitch_elems * es, batch_elems * es};
  cuuint32_t box[3] = {f32 ? 32u : 64u, box_rows, 1};     // 128 bytes wide either way
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, gdim, gstr, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D byte tensor {cols, rows, 1} with a {128, 128, 1} box and 128-byte swizzle (FP8 operands).
bool encode_map_u8(CUtensorMap* map, void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = get_encode_fn();
  if (!fn) return false;
  cuuint64_t gdim[3] = {cols, rows, 1};
  cuuint64_t gstr[2] = {pitch_bytes, pitch_bytes * rows};
  cuuint32_t box[3] = {128u, 128u, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, base, gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int check_launch(signmuon_ctx* c) {
  if (cudaGetLastError() != cudaSuccess) c->sticky = SIGNMUON_ERR_CUDA;
  return c->sticky;
}

// One-CTA tiles: `lists` CTAs.  CTA pairs: a cluster of two CTAs per tile list.
template <int BN, int STAGES, int EPI_BUFS, int CTAS, int KIND>
void launch_tc(const GemmLaunchArgs& a, int lists, cudaStream_t s) {
  constexpr size_t smem = ns_gemm_tc_smem_bytes<BN, STAGES, EPI_BUFS, CTAS, KIND>();
  if (CTAS == 1) {
    ns_gemm_tc_kernel<BN, STAGES, EPI_BUFS, CTAS, KIND><<<lists, GEMM_THREADS, smem, s>>>(a);
    return;
  }
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)lists * CTAS, 1, 1);
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = CTAS;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, ns_gemm_tc_kernel<BN, STAGES, EPI_BUFS, CTAS, KIND>, a);
}

// Shapes of the tensor-core kernel in use.  Gram launches have a long K loop and a small bf16 output:
// deep operand ring, two half-size output buffers.  Apply launches have a short K loop and move 8 bytes
// per entry through the epilogue: shallower operand ring, four chunk buffers (two C loads in flight).
// (BN, operand stages, chunk buffers, CTAs per tile, kind)
#define NS_GEMM_PAIR_GRAM 256, 5, 2, 2, 0
#define NS_GEMM_PAIR_APPLY 256, 4, 3, 2, 1
#define NS_GEMM_PAIR_APPLY_LONGK 256, 5, 2, 2, 1   /* long contraction: the operand ring matters more than the chunk ring */
#define NS_GEMM_ONE_GRAM 128, 5, 2, 1, 0
#define NS_GEMM_ONE_APPLY 128, 3, 4, 1, 1

template <int BN, int STAGES, int EPI_BUFS, int CTAS, int KIND>
bool opt_in_smem() {
  return cudaFuncSetAttribute(ns_gemm_tc_kernel<BN, STAGES, EPI_BUFS, CTAS, KIND>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)ns_gemm_tc_smem_bytes<BN, STAGES, EPI_BUFS, CTAS, KIND>()) == cudaSuccess;
}

// Opt in to the large dynamic shared memory of the tensor-core kernels (per device, at bind) and ask how
// many CTA pairs the device can hold at once.
bool configure_kernels(int* max_pairs) {
  bool ok = opt_in_smem<NS_GEMM_PAIR_GRAM>() && opt_in_smem<NS_GEMM_PAIR_APPLY>() && opt_in_smem<NS_GEMM_ONE_GRAM>() &&
            opt_in_smem<NS_GEMM_ONE_APPLY>() && opt_in_smem<NS_GEMM_PAIR_APPLY_LONGK>() &&
            cudaFuncSetAttribute(ns_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)CHAIN_SMEM_BYTES) == cudaSuccess;
  if (!ok) return false;
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = ns_gemm_tc_smem_bytes<NS_GEMM_PAIR_APPLY>();
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, ns_gemm_tc_kernel<NS_GEMM_PAIR_APPLY>, &cfg) != cudaSuccess || n < 1) return false;
  *max_pairs = n;
  return true;
}

// Device address of the parameter table of the step being enqueued.
const ParamDev* cur_paramdev(const signmuon_ctx* c) {
  return reinterpret_cast<const ParamDev*>(c->d_ws + c->off_paramdev + (size_t)c->cur_table * c->paramdev_stride);
}

void launch_gemm(signmuon_ctx* c, const LaunchPlan& lp, float lr, cudaStream_t s) {
  const TileTable& tt = c->tables[lp.tile_table];
  if (tt.tiles.empty()) return;
  const GemmProblem* probs = reinterpret_cast<const GemmProblem*>(c->d_ws + c->off_problems) + lp.problem_base;
  const TileEntry* tiles = reinterpret_cast<const TileEntry*>(c->d_ws + tt.tiles_off);
  const ParamDev* pd = cur_paramdev(c);
  if (c->cfg.flags & SIGNMUON_FLAG_SIMT_GEMM) {
    ns_gemm_simt_kernel<<<(unsigned)tt.tiles.size(), 128, 0, s>>>(probs, tiles, tt.bn, pd, lr, c->peers);
    return;
  }
  GemmLaunchArgs a;
  a.tmaps = reinterpret_cast<const CUtensorMap*>(c->d_ws + c->off_tmaps);
  a.problems = probs;
  a.tiles = tiles;
  a.cta_tile_start = reinterpret_cast<const uint32_t*>(c->d_ws + tt.cta_off);
  a.params = pd;
  a.status = reinterpret_cast<uint32_t*>(c->d_ws + c->off_status);
  a.lr = lr;
  a.wait_limit_ns = c->wait_limit_ns;
  a.peers = c->peers;
  const bool gram = lp.gram;
  if (tt.ctas == 2) {
    if (gram) launch_tc<NS_GEMM_PAIR_GRAM>(a, tt.grid, s);
    else if (tt.long_k) launch_tc<NS_GEMM_PAIR_APPLY_LONGK>(a, tt.grid, s);
    else launch_tc<NS_GEMM_PAIR_APPLY>(a, tt.grid, s);
  } else {
    if (gram) launch_tc<NS_GEMM_ONE_GRAM>(a, tt.grid, s); else launch_tc<NS_GEMM_ONE_APPLY>(a, tt.grid, s);
  }
}

// Vote over `rows` payload rows starting at `src` (default: all workers' rows of the payload buffer), then the
// update from the vote words.
// Gram-space chain of the parameters with a short side up to 256: one CTA pair per (parameter, worker) problem list.
void launch_chain(signmuon_ctx* c, int set, cudaStream_t s) {
  const signmuon_ctx::ChainSet& cs = c->chain[set];
  ChainLaunchArgs a;
  a.problems = reinterpret_cast<const ChainProblem*>(c->d_ws + cs.off_problems);
  a.order = reinterpret_cast<const uint32_t*>(c->d_ws + cs.off_order);
  a.pair_start = reinterpret_cast<const uint32_t*>(c->d_ws + cs.off_start);
  a.status = reinterpret_cast<uint32_t*>(c->d_ws + c->off_status);
  a.wait_limit_ns = c->wait_limit_ns;
  a.K = c->cfg.ns_steps;
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)cs.pairs * 2, 1, 1);
  cfg.blockDim = dim3(CHAIN_THREADS, 1, 1);
  cfg.dynamicSmemBytes = CHAIN_SMEM_BYTES;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, ns_chain_kernel, a);
}

template <int PLANES>
void launch_vote(signmuon_ctx* c, float lr, int write_sbar, cudaStream_t s, const uint32_t* src = nullptr, int rows = 0) {
  const ParamDev* pd = cur_paramdev(c);
  const int32_t* list = reinterpret_cast<const int32_t*>(c->d_ws + c->off_list_vote);
  uint32_t* vote = reinterpret_cast<uint32_t*>(c->d_ws + c->off_vote);
  const int n = (int)c->vote_list.size();
  if (src != vote)      // (vote words computed elsewhere: only the update remains)
    vote_kernel<PLANES><<<c->vote_blocks, VOTE_THREADS, 0, s>>>(
        c->vote_ranges, src ? rows : c->M_all, src ? src : reinterpret_cast<const uint32_t*>(c->d_ws + c->off_bits),
        vote, (int64_t)c->bits_pitch);
  // Programmatic dependent launch: the update grid may begin (and request its weight vectors) while the vote grid
  // drains; it waits for the vote grid's completion before it reads a vote word.
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(c->upd_blocks, 1, 1);
  cfg.blockDim = dim3(EW_THREADS, 1, 1);
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  const uint32_t* starts = reinterpret_cast<const uint32_t*>(c->d_ws + c->off_starts_upd);
  if (write_sbar)
    cudaLaunchKernelEx(&cfg, update_kernel<true>, pd, list, starts, n, c->Wm, lr, static_cast<const uint32_t*>(vote));
  else
    cudaLaunchKernelEx(&cfg, update_kernel<false>, pd, list, starts, n, c->Wm, lr, static_cast<const uint32_t*>(vote));
}

void invalidate_tables(signmuon_ctx* c) {
  for (int t = 0; t < PARAM_TABLES; ++t) c->table_key[t].clear();
}

// Selects (or fills) the device-side parameter table that holds this call's weight and gradient pointers.
int upload_params(signmuon_ctx* c, void* const* weights, const void* const* grads, cudaStream_t s) {
  const size_t n = c->params.size();
  for (size_t p = 0; p < n; ++p) {
    if (!weights[p] || !grads[p]) return SIGNMUON_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(weights[p]) & 15) || (reinterpret_cast<uintptr_t>(grads[p]) & 15))
      return SIGNMUON_ERR_MISALIGNED;
  }
  ++c->table_clock;
  for (int t = 0; t < PARAM_TABLES; ++t) {
    const std::vector<const void*>& key = c->table_key[t];
    if (key.size() != 2 * n) continue;
    bool same = true;
    for (size_t p = 0; p < n && same; ++p) same = key[p] == weights[p] && key[n + p] == grads[p];
    if (same) {
      c->cur_table = t;
      c->table_used[t] = c->table_clock;
      return SIGNMUON_OK;
    }
  }
  int victim = -1;
  for (int t = 0; t < PARAM_TABLES && victim < 0; ++t)
    if (c->table_key[t].empty()) victim = t;
  if (victim < 0) {
    victim = 0;
    for (int t = 1; t < PARAM_TABLES; ++t)
      if (c->table_used[t] < c->table_used[victim]) victim = t;
  }
  // miss: the least recently used slot takes this pointer set.  Its pinned mirror may still be the source of
  // the copy that filled the slot last time (long finished in practice): wait for that copy only.
  ParamDev* mirror = c->h_tables + (size_t)victim * n;
  if (cudaEventSynchronize(c->ev_table[victim]) != cudaSuccess) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
  std::vector<const void*>& key = c->table_key[victim];
  key.resize(2 * n);
  for (size_t p = 0; p < n; ++p) {
    mirror[p] = c->paramdev[p];
    mirror[p].W = weights[p];
    mirror[p].G = grads[p];
    key[p] = weights[p];
    key[n + p] = grads[p];
  }
  // Kernels of earlier steps that read this slot were enqueued on the caller's stream before this copy: a
  // context is used from one stream at a time, so the copy is ordered behind them.
  if (cudaMemcpyAsync(c->d_ws + c->off_paramdev + (size_t)victim * c->paramdev_stride, mirror, n * sizeof(ParamDev),
                      cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaEventRecord(c->ev_table[victim], s) != cudaSuccess) {
    key.clear();
    c->sticky = SIGNMUON_ERR_CUDA;
    return c->sticky;
  }
  c->cur_table = victim;
  c->table_used[victim] = c->table_clock;
  return SIGNMUON_OK;
}

// `vote_from_words`: the vote words were produced elsewhere (from all-reduced sign sums): the vote stage then only
// maps them to the update (a one-row "vote" over the vote words themselves).
int run_stages_impl(signmuon_ctx* c, int32_t mask, void* const* weights, const void* const* grads, float lr,
                    cudaStream_t s, bool vote_from_words = false) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  if (!weights || !grads) return SIGNMUON_ERR_INVALID_ARG;
  if ((mask & SIGNMUON_STAGE_MOMENTUM) && c->power_start_floats && !c->d_power_start) return SIGNMUON_ERR_NOT_BOUND;
  if (lr < 0.f) lr = c->cfg.lr;
  int rc = upload_params(c, weights, grads, s);
  if (rc != SIGNMUON_OK) return rc;
  const int M = c->Wm, K = c->cfg.ns_steps;      // M: batch slots of the matrix parameters (own workers; 1: Muon rule)
  const ParamDev* pd = cur_paramdev(c);
  uint32_t* bits = reinterpret_cast<uint32_t*>(c->d_ws + c->off_bits);
  uint32_t* vote = reinterpret_cast<uint32_t*>(c->d_ws + c->off_vote);
  const int nm = (int)c->matrix_list.size(), np = (int)c->plain_list.size();
  const float eps = c->cfg.eps;

  if (mask & SIGNMUON_STAGE_MOMENTUM) {
    if (nm) {
      momentum_kernel<<<c->mom_blocks, EW_THREADS, 0, s>>>(
          pd, reinterpret_cast<const int32_t*>(c->d_ws + c->off_list_matrix),
          reinterpret_cast<const uint32_t*>(c->d_ws + c->off_starts_mom), nm, c->cfg.momentum, c->cfg.weight_decay);
      const int32_t* mlist = reinterpret_cast<const int32_t*>(c->d_ws + c->off_list_matrix);
      if (c->power_start_floats) {
        // scale = spectral (Alg. 4): sigma from P rounds of power iteration on the momentum (Alg. 5)
        const uint32_t* xs = reinterpret_cast<const uint32_t*>(c->d_ws + c->off_starts_xv);
        const uint32_t* ts = reinterpret_cast<const uint32_t*>(c->d_ws + c->off_starts_xtu);
        pi_norm_kernel<<<nm * M, EW_THREADS, 0, s>>>(pd, mlist, M, PI_NORM_START, eps);
        for (int it = 0; it < c->cfg.power_iters; ++it) {
          pi_xv_kernel<<<c->xv_blocks, EW_THREADS, 0, s>>>(pd, mlist, xs, nm, eps);
          pi_norm_kernel<<<nm * M, EW_THREADS, 0, s>>>(pd, mlist, M, PI_NORM_U, eps);
          pi_xtu_kernel<<<c->xtu_blocks, EW_THREADS, 0, s>>>(pd, mlist, ts, nm, eps);
          pi_norm_kernel<<<nm * M, EW_THREADS, 0, s>>>(pd, mlist, M, PI_NORM_V, eps);
        }
        pi_xv_kernel<<<c->xv_blocks, EW_THREADS, 0, s>>>(pd, mlist, xs, nm, eps);
        pi_norm_kernel<<<nm * M, EW_THREADS, 0, s>>>(pd, mlist, M, PI_NORM_SIGMA, eps);
      } else {
        const int warps = nm * M;
        finalize_norms_kernel<<<(warps * 32 + 255) / 256, 256, 0, s>>>(pd, mlist, nm, M, eps);
      }
    }
    if (np) {
      plain_params_kernel<<<c->plain_blocks, EW_THREADS, 0, s>>>(
          pd, reinterpret_cast<const int32_t*>(c->d_ws + c->off_list_plain),
          reinterpret_cast<const uint32_t*>(c->d_ws + c->off_starts_plain), np, c->Lw, c->cfg.momentum,
          c->cfg.weight_decay, lr, bits + (size_t)c->w_off * c->bits_pitch, vote, (int64_t)c->bits_pitch,
          c->sharded ? 0 : 1, c->peers);
    }
  }
  if ((mask & SIGNMUON_STAGE_NS) && nm) {
    bool chain_done = c->chain[0].problems.empty();
    for (const LaunchPlan& lp : c->ns_launches) {
      if (!chain_done && lp.tile_table != TT_GRAM_FIRST) { launch_chain(c, 0, s); chain_done = true; }
      launch_gemm(c, lp, lr, s);
    }
    if (c->packfb_blocks) {
      pack_kernel<<<c->packfb_blocks, EW_THREADS, 0, s>>>(
          pd, reinterpret_cast<const int32_t*>(c->d_ws + c->off_list_packfb),
          reinterpret_cast<const uint32_t*>(c->d_ws + c->off_starts_packfb), (int)c->packfb_list.size(),
          K == 0 ? 1 : 0, bits + (size_t)c->w_off * c->bits_pitch, (int64_t)c->bits_pitch, c->peers);
    }
  }
  if ((mask & SIGNMUON_STAGE_NS) && c->peer_flags.n > 0) {
    // fused exchange: every payload word of this step is stored (here and in the peers' buffers): tell the peers
    ++c->exchange_seq;
    publish_payload_kernel<<<1, 32, 0, s>>>(c->peer_flags, c->my_rank, c->exchange_seq);
  }
  if ((mask & SIGNMUON_STAGE_VOTE) && c->peer_flags.n > 0) {
    // ... and wait (bounded) until every peer has told this GPU the same
    await_payloads_kernel<<<1, 64, 0, s>>>(reinterpret_cast<const uint32_t*>(c->d_ws + c->off_flags), c->n_ranks,
                                           c->my_rank, c->exchange_seq, c->wait_limit_ns,
                                           reinterpret_cast<uint32_t*>(c->d_ws + c->off_status));
  }
  const bool lp_ns = c->lp && K > 0;
  if ((mask & SIGNMUON_STAGE_VOTE) && !c->vote_list.empty()) {
    // local polar with K = 0 degenerates to S / ||S||_F: plain update with the Eq. 2 scale
    const int write_sbar = lp_ns ? 1 : 0;
    if (vote_from_words) launch_vote<3>(c, lr, write_sbar, s, vote, 1);      // update only
    else if (c->M_all <= 7) launch_vote<3>(c, lr, write_sbar, s);
    else if (c->M_all <= 63) launch_vote<6>(c, lr, write_sbar, s);
    else launch_vote<8>(c, lr, write_sbar, s);
  }
  if ((mask & SIGNMUON_STAGE_VOTE) && (c->cfg.flags & SIGNMUON_FLAG_SIGN_AGREEMENT)) {
    // after the vote of the matrix parameters (the plain parameters voted in the momentum stage)
    unsigned long long* agree = reinterpret_cast<unsigned long long*>(c->d_ws + c->off_agree);
    if (cudaMemsetAsync(agree, 0, (size_t)c->M_all * 8, s) != cudaSuccess) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
    const unsigned gx = (unsigned)std::min<uint64_t>((c->words_per_worker + EW_THREADS - 1) / EW_THREADS, 1024);
    sign_agreement_kernel<<<dim3(gx, (unsigned)c->M_all), EW_THREADS, 0, s>>>(bits, vote, (int64_t)c->words_per_worker,
                                                                             (int64_t)c->bits_pitch, agree);
  }
  if ((mask & SIGNMUON_STAGE_LOCAL_POLAR) && nm && lp_ns) {
    bool chain_done = c->chain[1].problems.empty();
    for (const LaunchPlan& lp : c->lp_launches) {
      if (!chain_done && lp.tile_table != TT_LP_GRAM_FIRST) { launch_chain(c, 1, s); chain_done = true; }
      launch_gemm(c, lp, lr, s);
    }
  }
  return check_launch(c);
}

}  // namespace

// =============================================================================== C ABI
extern "C" {

int signmuon_create(const signmuon_config* config, signmuon_ctx** out) {
  if (!out) return SIGNMUON_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config || config->num_params < 1 || !config->params) return SIGNMUON_ERR_INVALID_ARG;
  if (config->num_workers < 1 || config->num_workers > 255) return SIGNMUON_ERR_INVALID_ARG;
  if (!(config->momentum >= 0.f && config->momentum < 1.f)) return SIGNMUON_ERR_INVALID_ARG;
  if (config->ns_steps < 0 || config->ns_steps > 64) return SIGNMUON_ERR_INVALID_ARG;
  if (!(config->weight_decay >= 0.f)) return SIGNMUON_ERR_INVALID_ARG;
  if (!(config->lr == config->lr)) return SIGNMUON_ERR_INVALID_ARG;
  if (config->update_scale != 0 && config->update_scale != 1) return SIGNMUON_ERR_INVALID_ARG;
  if (config->local_polar != 0 && config->local_polar != 1) return SIGNMUON_ERR_INVALID_ARG;
  if (config->ns_scale != SIGNMUON_SCALE_FRO && config->ns_scale != SIGNMUON_SCALE_SPECTRAL) return SIGNMUON_ERR_INVALID_ARG;
  if (config->power_iters < 0 || config->power_iters > 64) return SIGNMUON_ERR_INVALID_ARG;
  if (config->local_workers < 0 || config->local_workers > config->num_workers) return SIGNMUON_ERR_INVALID_ARG;
  if (config->update_rule != SIGNMUON_RULE_SIGNMUON && config->update_rule != SIGNMUON_RULE_MUON) return SIGNMUON_ERR_INVALID_ARG;
  // Muon averages float gradients: with the workers on several GPUs that is the caller's all-reduce (then M = 1 here)
  if (config->update_rule == SIGNMUON_RULE_MUON && config->local_workers > 0 && config->local_workers < config->num_workers)
    return SIGNMUON_ERR_INVALID_ARG;
  if (config->update_rule == SIGNMUON_RULE_MUON && config->ns_steps == 0) return SIGNMUON_ERR_INVALID_ARG;   // the update lives in the last Newton-Schulz epilogue
  if (config->local_workers > 0 &&
      (config->worker_offset < 0 || config->worker_offset + config->local_workers > config->num_workers))
    return SIGNMUON_ERR_INVALID_ARG;
  for (int i = 0; i < config->num_params; ++i) {
    const signmuon_param& p = config->params[i];
    if (p.rows < 1 || p.cols < 1 || p.rows > (1 << 24) || p.cols > (1 << 24)) return SIGNMUON_ERR_BAD_SHAPE;
    if (p.kind != SIGNMUON_PARAM_MATRIX && p.kind != SIGNMUON_PARAM_PLAIN) return SIGNMUON_ERR_INVALID_ARG;
    if (!valid_dtype(p.weight_dtype) || !valid_dtype(p.grad_dtype)) return SIGNMUON_ERR_INVALID_ARG;
    if (p.kind == SIGNMUON_PARAM_MATRIX && std::min(p.rows, p.cols) > 65536 * 2) return SIGNMUON_ERR_BAD_SHAPE;
    // tile coordinates are 16-bit, in units of at least 128 rows or columns
    if (p.kind == SIGNMUON_PARAM_MATRIX && (std::max(p.rows, p.cols) + 127) / 128 > 65535) return SIGNMUON_ERR_BAD_SHAPE;
    if (p.rows * p.cols > (1ll << 36)) return SIGNMUON_ERR_BAD_SHAPE;
  }
  signmuon_ctx* c = new (std::nothrow) signmuon_ctx();
  if (!c) return SIGNMUON_ERR_NO_MEMORY;
  c->cfg = *config;
  if (!(c->cfg.eps > 0.f)) c->cfg.eps = 1e-12f;
  c->M_all = config->num_workers;
  c->Lw = config->local_workers > 0 ? config->local_workers : config->num_workers;
  c->w_off = config->local_workers > 0 ? config->worker_offset : 0;
  c->sharded = c->Lw < c->M_all;
  c->muon = config->update_rule == SIGNMUON_RULE_MUON;
  c->Wm = c->muon ? 1 : c->Lw;
  c->lp = config->local_polar != 0 && !c->muon;
  c->params.assign(config->params, config->params + config->num_params);
  c->cfg.params = nullptr;
  int rc = plan_layout(c);
  if (rc != SIGNMUON_OK) { delete c; return rc; }
  *out = c;
  return SIGNMUON_OK;
}

int signmuon_state_bytes(const signmuon_ctx* c, size_t* state, size_t* workspace, size_t* host_staging) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  if (state) *state = c->state_bytes;
  if (workspace) *workspace = c->workspace_bytes;
  if (host_staging) *host_staging = c->staging_bytes;
  return SIGNMUON_OK;
}

int signmuon_bind(signmuon_ctx* c, void* dev_state, size_t state_bytes, void* dev_workspace, size_t workspace_bytes,
                  void* dev_staging, size_t staging_bytes, int zero_state, void* cuda_stream) {
  if (!c || !dev_state || !dev_workspace) return SIGNMUON_ERR_INVALID_ARG;
  if (state_bytes < c->state_bytes || workspace_bytes < c->workspace_bytes) return SIGNMUON_ERR_BUFFER_TOO_SMALL;
  if (dev_staging && staging_bytes < c->staging_bytes) return SIGNMUON_ERR_BUFFER_TOO_SMALL;
  if ((reinterpret_cast<uintptr_t>(dev_state) & 255) || (reinterpret_cast<uintptr_t>(dev_workspace) & 1023) ||
      (reinterpret_cast<uintptr_t>(dev_staging) & 255))
    return SIGNMUON_ERR_MISALIGNED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  int dev = 0, major = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SIGNMUON_ERR_CUDA;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return SIGNMUON_ERR_CUDA;
  if (major != 10) return SIGNMUON_ERR_UNSUPPORTED_ARCH;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  c->num_sms = std::max(1, std::min(sms, MAX_CTAS));
  c->d_state = static_cast<uint8_t*>(dev_state);
  c->d_ws = static_cast<uint8_t*>(dev_workspace);
  c->d_staging = static_cast<uint8_t*>(dev_staging);
  if (dev_staging && !c->copy_stream) {
    bool sok = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 && sok; ++i) {
      sok = cudaEventCreateWithFlags(&c->ev_loaded[i], cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&c->ev_consumed[i], cudaEventDisableTiming) == cudaSuccess;
    }
    sok = sok && cudaEventCreateWithFlags(&c->ev_weights_up, cudaEventDisableTiming) == cudaSuccess;
    if (!sok) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
  }
  c->host_steps = 0;
  const int M = c->Wm;
  if (!c->h_tables) {   // pinned host mirrors of the parameter tables and the events that guard their reuse
    void* hp = nullptr;
    if (cudaHostAlloc(&hp, PARAM_TABLES * c->params.size() * sizeof(ParamDev), cudaHostAllocDefault) != cudaSuccess) {
      cudaGetLastError();
      return SIGNMUON_ERR_NO_MEMORY;
    }
    c->h_tables = static_cast<ParamDev*>(hp);
    for (int t = 0; t < PARAM_TABLES; ++t)
      if (cudaEventCreateWithFlags(&c->ev_table[t], cudaEventDisableTiming) != cudaSuccess) {
        c->sticky = SIGNMUON_ERR_CUDA;
        return c->sticky;
      }
  }

  // host image of the table area [0, off_tables_end) minus the big buffers: assemble piecewise
  auto up = [&](size_t off, const void* src, size_t bytes) -> bool {
    if (bytes == 0) return true;
    return cudaMemcpyAsync(c->d_ws + off, src, bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  };
  bool ok = cudaMemsetAsync(c->d_ws + c->off_status, 0, ALIGN, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->d_ws + c->off_flags, 0, 64 * 4, s) == cudaSuccess;
  c->peers.n = 0;            // peers are attached after bind (their addresses refer to bound buffers)
  c->peer_flags.n = 0;
  c->exchange_seq = 0;
  if (zero_state) ok = ok && cudaMemsetAsync(c->d_state, 0, c->state_bytes, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->d_ws + c->off_bits, 0, (size_t)c->M_all * c->bits_pitch * 4, s) == cudaSuccess;
  ok = ok && cudaMemsetAsync(c->d_ws + c->off_vote, 0, (size_t)c->bits_pitch * 4, s) == cudaSuccess;

  // parameter table (W/G filled in at the first step)
  c->paramdev.assign(c->params.size(), ParamDev());
  for (size_t p = 0; p < c->params.size(); ++p) {
    const ParamPlan& pl = c->plan[p];
    ParamDev& d = c->paramdev[p];
    std::memset(&d, 0, sizeof(d));
    d.mom = reinterpret_cast<float*>(c->d_state + pl.mom_off);
    if (pl.kind == SIGNMUON_PARAM_MATRIX) {
      d.y0 = reinterpret_cast<bf16*>(c->d_ws + pl.y_off[0]);
      d.y1 = reinterpret_cast<bf16*>(c->d_ws + pl.y_off[1]);
      d.ylo = (c->split || (pl.gs && !pl.gs_mem)) ? reinterpret_cast<bf16*>(c->d_ws + pl.lo_off[0]) : nullptr;
      d.yk_buf = pl.gs ? 1 : (c->cfg.ns_steps & 1);
      d.scales = reinterpret_cast<float*>(c->d_ws + pl.scales_off);
      d.partials = reinterpret_cast<float*>(c->d_ws + pl.partials_off);
      if (c->power_start_floats) {
        d.pi_v = reinterpret_cast<float*>(c->d_ws + pl.pi_v_off);
        d.pi_u = reinterpret_cast<float*>(c->d_ws + pl.pi_u_off);
        d.pi_scal = reinterpret_cast<float*>(c->d_ws + pl.pi_scal_off);
        d.pi_start = c->d_power_start ? c->d_power_start + pl.pi_start_off : nullptr;
      }
    }
    d.d = pl.d; d.rows = (int32_t)pl.rows; d.cols = (int32_t)pl.cols; d.ldy = pl.ldy;
    d.kind = pl.kind; d.wdtype = pl.wdtype; d.gdtype = pl.gdtype;
    d.word_off = pl.word_off; d.n_words = pl.n_words; d.chunks_per_worker = pl.chunks_per_worker;
    const bool eq2 = c->cfg.update_scale == 1 ||
                     (pl.kind == SIGNMUON_PARAM_MATRIX && c->lp && c->cfg.ns_steps == 0);
    d.upd_scale = eq2 ? (float)(1.0 / std::sqrt((double)pl.rows * (double)pl.cols)) : 1.f;
    d.vec_ok = (pl.d % 8 == 0 && pl.ldy == pl.cols) ? 1 : 0;
    d.avg_workers = (c->muon && pl.kind == SIGNMUON_PARAM_MATRIX) ? c->Lw : 1;
    d.sbar8 = pl.lp_fp8 ? c->d_ws + pl.s8_off : nullptr;
    d.ld8 = pl.ld8;
  }
  invalidate_tables(c);
  ok = ok && up(c->off_list_matrix, c->matrix_list.data(), c->matrix_list.size() * 4);
  ok = ok && up(c->off_list_plain, c->plain_list.data(), c->plain_list.size() * 4);
  ok = ok && up(c->off_list_packfb, c->packfb_list.data(), c->packfb_list.size() * 4);
  ok = ok && up(c->off_list_vote, c->vote_list.data(), c->vote_list.size() * 4);
  ok = ok && up(c->off_starts_mom, c->mom_starts.data(), c->mom_starts.size() * 4);
  ok = ok && up(c->off_starts_plain, c->plain_starts.data(), c->plain_starts.size() * 4);
  ok = ok && up(c->off_starts_upd, c->upd_starts.data(), c->upd_starts.size() * 4);
  ok = ok && up(c->off_starts_packfb, c->packfb_starts.data(), c->packfb_starts.size() * 4);
  ok = ok && up(c->off_starts_xv, c->xv_starts.data(), c->xv_starts.size() * 4);
  ok = ok && up(c->off_starts_xtu, c->xtu_starts.data(), c->xtu_starts.size() * 4);
  if (!ok) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }

  // tile tables (need the SM count) and tensor maps (need the device addresses)
  const size_t nm = c->matrix_list.size();
  int max_pairs = 1;
  if (!configure_kernels(&max_pairs)) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
  max_pairs = std::min(max_pairs, MAX_CTAS);
  for (int t = 0; t < TT_COUNT; ++t) {
    TileTable& tt = c->tables[t];
    tt.tiles.clear();
    tt.flops = 0;
    if (!tt.used) continue;
    build_tile_table(tt, c->problems, tt.problem_base, tt.problem_count, tt.ctas == 2 ? max_pairs : c->num_sms);
    ok = ok && up(tt.tiles_off, tt.tiles.data(), tt.tiles.size() * sizeof(TileEntry));
    ok = ok && up(tt.cta_off, tt.cta_start.data(), tt.cta_start.size() * 4);
    // Flops the tensor cores are asked for by one launch of this table: every scheduled tile issues whole
    // bm x bn x (128 bytes of K) blocks (ragged edges are zero-filled, skipped mirror tiles of the symmetric Gram
    // products are not issued at all), once per operand segment.
    for (const TileEntry& te : tt.tiles) {
      const GemmProblem& pr = c->problems[tt.problem_base + te.problem];
      const int kelem = pr.fp8 ? 2 * GEMM_BK : GEMM_BK;
      const double kblocks = (double)((pr.K + kelem - 1) / kelem) * (pr.nseg > 1 ? pr.nseg : 1);
      tt.flops += 2.0 * tt.bm * tt.bn * kelem * kblocks;
    }
  }
  c->executed_flops = 0;
  for (const LaunchPlan& lp : c->ns_launches) c->executed_flops += c->tables[lp.tile_table].flops;
  for (const LaunchPlan& lp : c->lp_launches) c->executed_flops += c->tables[lp.tile_table].flops;
  // chain launches: problems to CTA pairs, longest first (cost ~ s^2: contraction steps x columns walked)
  for (int set = 0; set < 2; ++set) {
    signmuon_ctx::ChainSet& cs = c->chain[set];
    cs.pairs = 0;
    if (cs.problems.empty()) continue;
    const int K = c->cfg.ns_steps;
    std::vector<ChainProblem> cps = cs.problems;
    std::vector<uint32_t> idx(cps.size());
    for (size_t i = 0; i < cps.size(); ++i) {
      idx[i] = (uint32_t)i;
      cps[i].q_hi = reinterpret_cast<bf16*>(c->d_ws + reinterpret_cast<size_t>(cps[i].q_hi));
      cps[i].q_lo = reinterpret_cast<bf16*>(c->d_ws + reinterpret_cast<size_t>(cps[i].q_lo));
      // products of the chain: A A and A (A A) in every iteration but the last, A F in every iteration but the first
      c->executed_flops += 3.0 * (K - 1) * 2.0 * 256.0 * 256.0 * (double)(((cps[i].s + 15) / 16) * 16);
    }
    std::stable_sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) { return cps[a].s > cps[b].s; });
    cs.pairs = (int)std::min<size_t>((size_t)max_pairs, cps.size());
    std::vector<std::vector<uint32_t>> per((size_t)cs.pairs);
    typedef std::pair<long long, int> Load;
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int i = 0; i < cs.pairs; ++i) heap.push({0, i});
    for (uint32_t i : idx) {
      Load top = heap.top();
      heap.pop();
      per[top.second].push_back(i);
      heap.push({top.first + (long long)cps[i].s * cps[i].s + 4096, top.second});
    }
    std::vector<uint32_t> order, pair_start((size_t)cs.pairs + 1, 0);
    for (int i = 0; i < cs.pairs; ++i) {
      pair_start[i] = (uint32_t)order.size();
      order.insert(order.end(), per[i].begin(), per[i].end());
    }
    pair_start[cs.pairs] = (uint32_t)order.size();
    ok = ok && up(cs.off_problems, cps.data(), cps.size() * sizeof(ChainProblem));
    ok = ok && up(cs.off_order, order.data(), order.size() * 4);
    ok = ok && up(cs.off_start, pair_start.data(), pair_start.size() * 4);
    ok = ok && cudaStreamSynchronize(s) == cudaSuccess;      // (the host vectors die with this scope)
  }
  std::vector<CUtensorMap> maps((size_t)c->num_tmaps);
  const bool need_maps = !(c->cfg.flags & SIGNMUON_FLAG_SIMT_GEMM) && c->cfg.ns_steps > 0;
  if (need_maps) {
    for (int32_t p : c->matrix_list) {
      const ParamPlan& pl = c->plan[p];
      CUtensorMap* mp = maps.data() + pl.tmap_base;
      const uint32_t bn = 128;   // box rows of a K-major B operand = tile width
      const uint64_t slots = (uint64_t)M + (c->lp ? 1 : 0);
      for (int buf = 0; buf < 2; ++buf) {
        void* y = c->d_ws + pl.y_off[buf];
        const uint64_t yb = (uint64_t)pl.rows * pl.ldy;
        ok = ok && encode_map(mp + buf * 3 + 0, y, pl.cols, pl.rows, slots, pl.ldy, yb, 128);
        ok = ok && encode_map(mp + buf * 3 + 1, y, pl.cols, pl.rows, slots, pl.ldy, yb, bn);
        ok = ok && encode_map(mp + buf * 3 + 2, y, pl.cols, pl.rows, slots, pl.ldy, yb, 64);
      }
      void* q = c->d_ws + pl.q_off;
      const uint64_t qb = (uint64_t)pl.s * pl.ldq;
      ok = ok && encode_map(mp + TM_Q_K128, q, pl.s, pl.s, slots, pl.ldq, qb, 128);
      ok = ok && encode_map(mp + TM_Q_KBN, q, pl.s, pl.s, slots, pl.ldq, qb, bn);
      ok = ok && encode_map(mp + TM_Q_BOX64, q, pl.s, pl.s, slots, pl.ldq, qb, 64);
      for (int b2 = 0; b2 < 2; ++b2) {
        ok = ok && encode_map(mp + (b2 ? TM_LO1_K128 : TM_LO0_K128), c->d_ws + pl.lo_off[b2], pl.cols, pl.rows, slots,
                              pl.ldy, (uint64_t)pl.rows * pl.ldy, 128);
        ok = ok && encode_map(mp + (b2 ? TM_LO1_MN : TM_LO0_MN), c->d_ws + pl.lo_off[b2], pl.cols, pl.rows, slots,
                              pl.ldy, (uint64_t)pl.rows * pl.ldy, 64);
      }
      if (c->split || pl.gs) {
        ok = ok && encode_map(mp + TM_QLO_K128, c->d_ws + pl.qlo_off, pl.s, pl.s, slots, pl.ldq, qb, 128);
        ok = ok && encode_map(mp + TM_QLO_KBN, c->d_ws + pl.qlo_off, pl.s, pl.s, slots, pl.ldq, qb, bn);
      }
      if (pl.gs_mem) {
        const size_t offs[7] = {pl.gc_q1_off, pl.gc_q1lo_off, pl.gc_r_off, pl.gc_h_off[0], pl.gc_hlo_off[0], pl.gc_h_off[1],
                                pl.gc_hlo_off[1]};
        for (int i = 0; i < 7; ++i)
          ok = ok && encode_map(mp + TM_GC_Q1 + i, c->d_ws + offs[i], pl.s, pl.s, slots, pl.ldq, qb, 128);
      }
      if (pl.lp_fp8)          // FP8 copy of the vote matrix: {128 bytes x 128 rows} boxes serve K-major and MN-major tiles
        ok = ok && encode_map_u8(mp + TM_S8, c->d_ws + pl.s8_off, pl.cols, pl.rows, pl.ld8);
      if (pl.cols % 4 == 0)   // float32 momentum as the first iteration's C operand
        ok = ok && encode_map(mp + TM_MOM_F32, c->d_state + pl.mom_off, pl.cols, pl.rows, M, pl.cols, (uint64_t)pl.d, 128,
                              true);
    }
    if (!ok) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
    ok = ok && up(c->off_tmaps, maps.data(), maps.size() * sizeof(CUtensorMap));
  }
  // resolve workspace-relative pointers of the problems
  std::vector<GemmProblem> probs = c->problems;
  for (GemmProblem& pr : probs) {
    pr.A = reinterpret_cast<const bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.A));
    pr.B = reinterpret_cast<const bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.B));
    pr.out = c->d_ws + reinterpret_cast<size_t>(pr.out);
    if (pr.epi != EPI_GRAM) {
      uint8_t* cbase = (pr.c_mode == C_F32) ? c->d_state : c->d_ws;
      pr.C = cbase + reinterpret_cast<size_t>(pr.C);
      if (pr.C_lo) pr.C_lo = reinterpret_cast<const bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.C_lo));
      if (pr.c2_coef != 0.f) {
        pr.C2 = reinterpret_cast<const bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.C2));
        pr.C2_lo = reinterpret_cast<const bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.C2_lo));
      }
      pr.out_lo = reinterpret_cast<bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.out_lo));
    } else if (pr.gram_lo) {
      pr.out_lo = reinterpret_cast<bf16*>(c->d_ws + reinterpret_cast<size_t>(pr.out_lo));
    }
    if (pr.scale_ptr) pr.scale_ptr = reinterpret_cast<const float*>(c->d_ws + reinterpret_cast<size_t>(pr.scale_ptr));
    if (pr.epi == EPI_APPLY_PACK)
      pr.bits_out = reinterpret_cast<uint32_t*>(c->d_ws + c->off_bits + reinterpret_cast<size_t>(pr.bits_out));
  }
  ok = ok && up(c->off_problems, probs.data(), probs.size() * sizeof(GemmProblem));
  // the uploads above read host vectors that die with this call: make sure they are consumed
  ok = ok && cudaStreamSynchronize(s) == cudaSuccess;
  if (!ok) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
  c->bound = true;
  c->sticky = SIGNMUON_OK;
  return SIGNMUON_OK;
}

int signmuon_step(signmuon_ctx* c, void* const* weights, const void* const* grads, float lr, void* cuda_stream) {
  if (c && c->sharded) return SIGNMUON_ERR_INVALID_ARG;   // the payload exchange belongs between the stages
  return run_stages_impl(c, SIGNMUON_STAGE_ALL, weights, grads, lr, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int signmuon_run_stages(signmuon_ctx* c, int32_t stage_mask, void* const* weights, const void* const* grads, float lr,
                        void* cuda_stream) {
  if (stage_mask & ~SIGNMUON_STAGE_ALL) return SIGNMUON_ERR_INVALID_ARG;
  return run_stages_impl(c, stage_mask, weights, grads, lr, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int signmuon_step_host(signmuon_ctx* c, void* const* host_weights, const void* const* host_grads, float lr,
                       void* cuda_stream) {
  if (!c || !host_weights || !host_grads) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound || !c->d_staging) return SIGNMUON_ERR_NOT_BOUND;
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int M = c->Lw;
  const size_t n = c->params.size();
  if (c->sharded) return SIGNMUON_ERR_INVALID_ARG;     // the exchange sits between the stages: see signmuon_step
  for (size_t p = 0; p < n; ++p)
    if (!host_weights[p] || !host_grads[p]) return SIGNMUON_ERR_INVALID_ARG;
  const int set = (int)(c->host_steps & 1);
  uint8_t* gbase = c->d_staging + c->stage_g_base + (size_t)set * c->stage_g_set_bytes;
  std::vector<void*> w(n);
  std::vector<const void*> g(n);
  bool ok = true;
  // gradients: internal stream, as soon as the step that last used this set (two calls ago) has finished
  if (c->host_steps >= 2) ok = cudaStreamWaitEvent(c->copy_stream, c->ev_consumed[set], 0) == cudaSuccess;
  // ... and behind the previous call's weight upload: that (small) copy becomes ready at the same moment as this
  // (large) one - when the step before it ends - and must not queue behind it in the host-to-device copy engine, or the
  // previous call's step would wait for this call's gradients
  if (c->host_steps >= 1) ok = ok && cudaStreamWaitEvent(c->copy_stream, c->ev_weights_up, 0) == cudaSuccess;
  for (size_t p = 0; p < n && ok; ++p) {
    const ParamPlan& pl = c->plan[p];
    g[p] = gbase + pl.stage_g_off;
    ok = cudaMemcpyAsync(const_cast<void*>(g[p]), host_grads[p], (size_t)M * pl.d * dtype_size(pl.gdtype),
                         cudaMemcpyHostToDevice, c->copy_stream) == cudaSuccess;
  }
  ok = ok && cudaEventRecord(c->ev_loaded[set], c->copy_stream) == cudaSuccess;
  // Weights.  Nothing before the vote stage touches them unless there are plain parameters (updated in the momentum
  // stage), coupled weight decay (read there) or the Muon rule (updated by the last Newton-Schulz epilogue): then they
  // too travel on the library's stream, behind the gradients and behind the previous call's copy back to the same
  // host arrays, and only the vote stage waits for them.  Otherwise they go first, on the caller's stream.
  const bool late_weights = c->plain_list.empty() && c->cfg.weight_decay == 0.f && !c->muon;
  cudaStream_t ws = late_weights ? c->copy_stream : s;
  if (late_weights && c->host_steps >= 1) ok = ok && cudaStreamWaitEvent(ws, c->ev_consumed[set ^ 1], 0) == cudaSuccess;
  for (size_t p = 0; p < n && ok; ++p) {
    const ParamPlan& pl = c->plan[p];
    w[p] = c->d_staging + pl.stage_w_off;
    ok = cudaMemcpyAsync(w[p], host_weights[p], (size_t)pl.d * dtype_size(pl.wdtype), cudaMemcpyHostToDevice, ws) == cudaSuccess;
  }
  ok = ok && cudaEventRecord(c->ev_weights_up, ws) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(s, c->ev_loaded[set], 0) == cudaSuccess;
  if (!ok) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
  int rc;
  if (late_weights) {
    rc = run_stages_impl(c, SIGNMUON_STAGE_MOMENTUM | SIGNMUON_STAGE_NS, w.data(), g.data(), lr, s);
    if (rc != SIGNMUON_OK) return rc;
    if (cudaStreamWaitEvent(s, c->ev_weights_up, 0) != cudaSuccess) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
    rc = run_stages_impl(c, SIGNMUON_STAGE_VOTE | SIGNMUON_STAGE_LOCAL_POLAR, w.data(), g.data(), lr, s);
  } else {
    rc = run_stages_impl(c, SIGNMUON_STAGE_ALL, w.data(), g.data(), lr, s);
  }
  if (rc != SIGNMUON_OK) return rc;
  for (size_t p = 0; p < n && ok; ++p) {
    const ParamPlan& pl = c->plan[p];
    ok = cudaMemcpyAsync(host_weights[p], w[p], (size_t)pl.d * dtype_size(pl.wdtype), cudaMemcpyDeviceToHost, s) == cudaSuccess;
  }
  ok = ok && cudaEventRecord(c->ev_consumed[set], s) == cudaSuccess;
  if (!ok) { c->sticky = SIGNMUON_ERR_CUDA; return c->sticky; }
  ++c->host_steps;
  return SIGNMUON_OK;
}

int signmuon_packed_payload(const signmuon_ctx* c, int32_t worker, const uint32_t** dev_ptr, size_t* bytes,
                            size_t* entries) {
  if (!c || worker < 0 || worker >= c->cfg.num_workers) return SIGNMUON_ERR_INVALID_ARG;
  if (bytes) *bytes = (size_t)c->words_per_worker * 4;
  if (entries) *entries = (size_t)c->entries;
  if (dev_ptr) {
    if (!c->bound) { *dev_ptr = nullptr; return SIGNMUON_ERR_NOT_BOUND; }
    *dev_ptr = reinterpret_cast<const uint32_t*>(c->d_ws + c->off_bits) + (size_t)worker * c->bits_pitch;
  }
  return SIGNMUON_OK;
}

int signmuon_payload_buffer(const signmuon_ctx* c, uint32_t** dev_ptr, size_t* row_pitch_bytes, int32_t* rows) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  if (row_pitch_bytes) *row_pitch_bytes = (size_t)c->bits_pitch * 4;
  if (rows) *rows = c->M_all;
  if (dev_ptr) {
    if (!c->bound) { *dev_ptr = nullptr; return SIGNMUON_ERR_NOT_BOUND; }
    *dev_ptr = reinterpret_cast<uint32_t*>(c->d_ws + c->off_bits);
  }
  return SIGNMUON_OK;
}

int signmuon_exchange_flags(const signmuon_ctx* c, uint32_t** dev_ptr) {
  if (!c || !dev_ptr) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) { *dev_ptr = nullptr; return SIGNMUON_ERR_NOT_BOUND; }
  *dev_ptr = reinterpret_cast<uint32_t*>(c->d_ws + c->off_flags);
  return SIGNMUON_OK;
}

int signmuon_set_payload_peers(signmuon_ctx* c, int32_t my_rank, int32_t num_ranks, int32_t num_peers,
                               uint32_t* const* peer_payload_buffers, uint32_t* const* peer_flags) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (num_peers < 0 || num_peers > MAX_PAYLOAD_PEERS || num_ranks < 1 || num_ranks > 64 || my_rank < 0 ||
      my_rank >= num_ranks || num_peers >= num_ranks + (num_peers == 0 ? 1 : 0))
    return SIGNMUON_ERR_INVALID_ARG;
  if (num_peers > 0 && (!peer_payload_buffers || !peer_flags)) return SIGNMUON_ERR_INVALID_ARG;
  PeerList pl = {};
  FlagList fl = {};
  const char* own = reinterpret_cast<const char*>(c->d_ws + c->off_bits);
  for (int p = 0; p < num_peers; ++p) {
    if (!peer_payload_buffers[p] || !peer_flags[p]) return SIGNMUON_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(peer_payload_buffers[p]) & 127) || (reinterpret_cast<uintptr_t>(peer_flags[p]) & 3))
      return SIGNMUON_ERR_MISALIGNED;
    pl.delta[p] = reinterpret_cast<const char*>(peer_payload_buffers[p]) - own;
    fl.flags[p] = peer_flags[p];
  }
  pl.n = fl.n = num_peers;
  c->peers = pl;
  c->peer_flags = fl;
  c->my_rank = my_rank;
  c->n_ranks = num_ranks;
  return SIGNMUON_OK;
}

int signmuon_vote_update(signmuon_ctx* c, const uint32_t* const* payloads, void* const* weights,
                         const void* const* grads, float lr, void* cuda_stream) {
  if (!c || !payloads) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint32_t* rows = reinterpret_cast<uint32_t*>(c->d_ws + c->off_bits);
  for (int m = 0; m < c->M_all; ++m) {
    const uint32_t* src = payloads[m];
    uint32_t* dst = rows + (size_t)m * c->bits_pitch;
    if (!src || src == dst) continue;
    if (reinterpret_cast<uintptr_t>(src) & 3) return SIGNMUON_ERR_MISALIGNED;
    if (cudaMemcpyAsync(dst, src, (size_t)c->words_per_worker * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess) {
      c->sticky = SIGNMUON_ERR_CUDA;
      return c->sticky;
    }
  }
  return run_stages_impl(c, SIGNMUON_STAGE_VOTE | SIGNMUON_STAGE_LOCAL_POLAR, weights, grads, lr, s);
}

int signmuon_local_sign_sum(signmuon_ctx* c, int8_t* dev_sums, size_t bytes, void* cuda_stream) {
  if (!c || !dev_sums) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  if (c->M_all > 127) return SIGNMUON_ERR_INVALID_ARG;              // the reduced sums must fit int8
  if (bytes < (size_t)c->words_per_worker * 32) return SIGNMUON_ERR_BUFFER_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(dev_sums) & 15) return SIGNMUON_ERR_MISALIGNED;
  const uint32_t* rows = reinterpret_cast<const uint32_t*>(c->d_ws + c->off_bits) + (size_t)c->w_off * c->bits_pitch;
  const unsigned blocks = (unsigned)((c->words_per_worker + EW_THREADS - 1) / EW_THREADS);
  sign_sum_kernel<<<blocks, EW_THREADS, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      rows, (int64_t)c->bits_pitch, (int64_t)c->words_per_worker, c->Lw, dev_sums);
  return check_launch(c);
}

int signmuon_vote_update_from_sums(signmuon_ctx* c, const int8_t* dev_sums, size_t bytes, void* const* weights,
                                   const void* const* grads, float lr, void* cuda_stream) {
  if (!c || !dev_sums) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  if (bytes < (size_t)c->words_per_worker * 32) return SIGNMUON_ERR_BUFFER_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(dev_sums) & 15) return SIGNMUON_ERR_MISALIGNED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  const unsigned blocks = (unsigned)((c->words_per_worker + EW_THREADS - 1) / EW_THREADS);
  sums_to_vote_kernel<<<blocks, EW_THREADS, 0, s>>>(dev_sums, (int64_t)c->words_per_worker,
                                                    reinterpret_cast<uint32_t*>(c->d_ws + c->off_vote));
  return run_stages_impl(c, SIGNMUON_STAGE_VOTE | SIGNMUON_STAGE_LOCAL_POLAR, weights, grads, lr, s, true);
}

int signmuon_payload_segment(const signmuon_ctx* c, int32_t param, size_t* word_offset, size_t* words) {
  if (!c || param < 0 || param >= (int32_t)c->params.size()) return SIGNMUON_ERR_INVALID_ARG;
  if (word_offset) *word_offset = c->plan[param].word_off;
  if (words) *words = c->plan[param].n_words;
  return SIGNMUON_OK;
}

int signmuon_debug_tap(const signmuon_ctx* c, int32_t what, int32_t param, int32_t worker, const void** dev_ptr,
                       size_t* bytes, int64_t* ld) {
  if (!c || !dev_ptr || param < 0 || param >= (int32_t)c->params.size()) return SIGNMUON_ERR_INVALID_ARG;
  if (worker < 0 || worker >= c->cfg.num_workers) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  const ParamPlan& pl = c->plan[param];
  // momentum, Y_K and norm factors exist for this context's own workers only
  const bool own = worker >= c->w_off && worker < c->w_off + c->Lw;
  if (!own && (what == SIGNMUON_TAP_MOMENTUM || what == SIGNMUON_TAP_POLAR || what == SIGNMUON_TAP_NORM))
    return SIGNMUON_ERR_INVALID_ARG;
  const int32_t lw = worker - c->w_off;                 // index among the own workers
  if (c->muon && pl.kind == SIGNMUON_PARAM_MATRIX) {    // one momentum, nothing packed or voted
    if (what != SIGNMUON_TAP_MOMENTUM && what != SIGNMUON_TAP_NORM) return SIGNMUON_ERR_INVALID_ARG;
    if (lw != 0) return SIGNMUON_ERR_INVALID_ARG;
  }
  size_t nbytes = 0;
  int64_t pitch = pl.cols;
  const void* ptr = nullptr;
  switch (what) {
    case SIGNMUON_TAP_MOMENTUM:
      ptr = c->d_state + pl.mom_off + (size_t)lw * pl.d * 4; nbytes = (size_t)pl.d * 4; break;
    case SIGNMUON_TAP_POLAR: {
      if (pl.kind != SIGNMUON_PARAM_MATRIX) return SIGNMUON_ERR_INVALID_ARG;
      if (!(c->cfg.flags & SIGNMUON_FLAG_KEEP_POLAR) && pl.fused_pack) return SIGNMUON_ERR_INVALID_ARG;
      const size_t yb = (size_t)pl.rows * pl.ldy * 2;
      ptr = c->d_ws + pl.y_off[pl.gs ? 1 : (c->cfg.ns_steps & 1)] + (size_t)lw * yb; nbytes = yb; pitch = pl.ldy; break;
    }
    case SIGNMUON_TAP_VOTE_BITS:
      ptr = c->d_ws + c->off_vote + (size_t)pl.word_off * 4; nbytes = (size_t)pl.n_words * 4; break;
    case SIGNMUON_TAP_WORKER_BITS:
      ptr = c->d_ws + c->off_bits + ((size_t)worker * c->bits_pitch + pl.word_off) * 4;
      nbytes = (size_t)pl.n_words * 4; break;
    case SIGNMUON_TAP_NORM:
      if (pl.kind != SIGNMUON_PARAM_MATRIX) return SIGNMUON_ERR_INVALID_ARG;
      ptr = c->d_ws + pl.scales_off + (size_t)lw * 8; nbytes = 8; break;
    default: return SIGNMUON_ERR_INVALID_ARG;
  }
  *dev_ptr = ptr;
  if (bytes) *bytes = nbytes;
  if (ld) *ld = pitch;
  return SIGNMUON_OK;
}

int signmuon_status(signmuon_ctx* c, void* cuda_stream) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, c->d_ws + c->off_status, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) {
    c->sticky = SIGNMUON_ERR_CUDA;
    return c->sticky;
  }
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  return word == STATUS_OK ? SIGNMUON_OK : SIGNMUON_ERR_TIMEOUT;
}

int signmuon_set_wait_limit(signmuon_ctx* c, uint64_t limit_ns) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  c->wait_limit_ns = limit_ns ? limit_ns : DEFAULT_WAIT_LIMIT_NS;
  return SIGNMUON_OK;
}

int signmuon_selftest_wait_timeout(signmuon_ctx* c, uint64_t limit_ns, void* cuda_stream) {
  if (!c || limit_ns == 0 || limit_ns > DEFAULT_WAIT_LIMIT_NS) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (c->sticky != SIGNMUON_OK) return c->sticky;
  wait_timeout_probe_kernel<<<1, 32, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(
      reinterpret_cast<uint32_t*>(c->d_ws + c->off_status), limit_ns);
  return check_launch(c);
}

int signmuon_power_start_size(const signmuon_ctx* c, size_t* floats) {
  if (!c || !floats) return SIGNMUON_ERR_INVALID_ARG;
  *floats = c->power_start_floats;
  return SIGNMUON_OK;
}

int signmuon_power_start_segment(const signmuon_ctx* c, int32_t param, size_t* float_offset, size_t* floats_per_worker) {
  if (!c || param < 0 || param >= (int32_t)c->params.size()) return SIGNMUON_ERR_INVALID_ARG;
  if (c->plan[param].kind != SIGNMUON_PARAM_MATRIX || c->power_start_floats == 0) return SIGNMUON_ERR_INVALID_ARG;
  if (float_offset) *float_offset = c->plan[param].pi_start_off;
  if (floats_per_worker) *floats_per_worker = (size_t)c->plan[param].cols;
  return SIGNMUON_OK;
}

int signmuon_set_power_start(signmuon_ctx* c, const float* dev_vectors, size_t floats) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  if (c->power_start_floats == 0) return SIGNMUON_ERR_INVALID_ARG;
  if (!dev_vectors) return SIGNMUON_ERR_INVALID_ARG;
  if (floats < c->power_start_floats) return SIGNMUON_ERR_BUFFER_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(dev_vectors) & 15) return SIGNMUON_ERR_MISALIGNED;
  if (c->d_power_start != dev_vectors) {
    c->d_power_start = dev_vectors;
    for (int32_t p : c->matrix_list) c->paramdev[p].pi_start = dev_vectors + c->plan[p].pi_start_off;
    invalidate_tables(c);             // every cached table goes to the device again when it is next used
  }
  return SIGNMUON_OK;
}

int signmuon_sign_agreement(signmuon_ctx* c, uint64_t* host_agree, uint64_t* host_entries, void* cuda_stream) {
  if (!c || !host_agree) return SIGNMUON_ERR_INVALID_ARG;
  if (!(c->cfg.flags & SIGNMUON_FLAG_SIGN_AGREEMENT)) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int M = c->M_all;
  std::vector<unsigned long long> raw((size_t)M);
  if (cudaMemcpyAsync(raw.data(), c->d_ws + c->off_agree, (size_t)M * 8, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess) {
    c->sticky = SIGNMUON_ERR_CUDA;
    return c->sticky;
  }
  const uint64_t pads = c->words_per_worker * 32 - (uint64_t)c->entries;   // zero in every payload and in the vote
  for (int m = 0; m < M; ++m) host_agree[m] = (uint64_t)raw[m] - pads;
  if (host_entries) *host_entries = (uint64_t)c->entries;
  return SIGNMUON_OK;
}

int signmuon_launches_per_step(const signmuon_ctx* c, int32_t* launches) {
  if (!c || !launches) return SIGNMUON_ERR_INVALID_ARG;
  int n = 0;
  const bool nm = !c->matrix_list.empty();
  if (nm) n += 1 + (c->power_start_floats ? 3 + 4 * c->cfg.power_iters : 1);   // momentum + norms (or power iteration)
  if (!c->plain_list.empty()) n += 1;
  if (nm) n += (int)c->ns_launches.size() + (c->packfb_blocks ? 1 : 0);       // NS, fallback pack
  if (!c->chain[0].problems.empty()) n += 1;                                  // Gram-space chain
  if (!c->vote_list.empty()) n += 2;                                          // vote, update
  if (nm && c->lp && c->cfg.ns_steps > 0) n += (int)c->lp_launches.size() + (c->chain[1].problems.empty() ? 0 : 1);
  if (c->peer_flags.n > 0) n += 2;                                            // publish, await (fused exchange)
  if (c->cfg.flags & SIGNMUON_FLAG_SIGN_AGREEMENT) n += 1;
  *launches = n;
  return SIGNMUON_OK;
}

int signmuon_ns_flops_per_step(const signmuon_ctx* c, double* flops) {
  if (!c || !flops) return SIGNMUON_ERR_INVALID_ARG;
  double f = 0;
  for (int32_t p : c->matrix_list) {
    const ParamPlan& pl = c->plan[p];
    f += 4.0 * (double)pl.s * (double)pl.s * (double)pl.l * c->cfg.ns_steps *
         (c->Wm + (c->lp ? 1 : 0));
  }
  *flops = f;
  return SIGNMUON_OK;
}

int signmuon_ns_launches_per_step(const signmuon_ctx* c, int32_t* gemm_launches, int32_t* chain_launches) {
  if (!c) return SIGNMUON_ERR_INVALID_ARG;
  const bool lp = !c->matrix_list.empty() && c->lp && c->cfg.ns_steps > 0;
  if (gemm_launches) *gemm_launches = (int32_t)(c->ns_launches.size() + (lp ? c->lp_launches.size() : 0));
  if (chain_launches)
    *chain_launches = (c->chain[0].problems.empty() ? 0 : 1) + ((lp && !c->chain[1].problems.empty()) ? 1 : 0);
  return SIGNMUON_OK;
}

int signmuon_ns_executed_flops_per_step(const signmuon_ctx* c, double* flops) {
  if (!c || !flops) return SIGNMUON_ERR_INVALID_ARG;
  if (!c->bound) return SIGNMUON_ERR_NOT_BOUND;
  *flops = c->executed_flops;
  return SIGNMUON_OK;
}

void signmuon_destroy(signmuon_ctx* c) {
  if (!c) return;
  if (c->copy_stream) {
    cudaStreamSynchronize(c->copy_stream);
    for (int i = 0; i < 2; ++i) {
      if (c->ev_loaded[i]) cudaEventDestroy(c->ev_loaded[i]);
      if (c->ev_consumed[i]) cudaEventDestroy(c->ev_consumed[i]);
    }
    if (c->ev_weights_up) cudaEventDestroy(c->ev_weights_up);
    cudaStreamDestroy(c->copy_stream);
  }
  for (int t = 0; t < PARAM_TABLES; ++t)
    if (c->ev_table[t]) { cudaEventSynchronize(c->ev_table[t]); cudaEventDestroy(c->ev_table[t]); }
  if (c->h_tables) cudaFreeHost(c->h_tables);
  delete c;
}

const char* signmuon_error_string(int code) {
  switch (code) {
    case SIGNMUON_OK: return "ok";
    case SIGNMUON_ERR_INVALID_ARG: return "invalid argument";
    case SIGNMUON_ERR_BAD_SHAPE: return "bad parameter shape";
    case SIGNMUON_ERR_NOT_BOUND: return "context has no device buffers bound";
    case SIGNMUON_ERR_BUFFER_TOO_SMALL: return "state, workspace or staging buffer too small";
    case SIGNMUON_ERR_CUDA: return "CUDA call or kernel launch failed";
    case SIGNMUON_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case SIGNMUON_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
    case SIGNMUON_ERR_MISALIGNED: return "device pointer is not sufficiently aligned";
    case SIGNMUON_ERR_TOO_LARGE: return "problem exceeds the fixed capacity of this entry point";
    case SIGNMUON_ERR_NO_MEMORY: return "host memory allocation failed";
    default: return "unknown error";
  }
}

}  // extern "C"
