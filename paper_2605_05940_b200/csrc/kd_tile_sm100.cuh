// Fused LM-head tile kernel of the distillation step.
//
// For a block of 128 compact rows (the tokens that carry loss, numbered in packed order) and a
// run of 256-wide vocabulary tiles it forms the student logits O_S = H W^T (Algorithm 1,
// "Compute Student Logits") on tcgen05 tensor cores with the accumulator in tensor memory,
// streams the matching teacher-logit tile O_T through shared memory with TMA, and consumes
// both on chip.  The T x V logits are never written to global memory.
//
//   kForward : online softmax statistics of Softmax(O_T/tau) and Softmax(O_S/tau)
//              (Algorithm 1, "Compute Probs") and the cross term of Eq. 2, kept
//              as running (max, sum, sum*(difference)) per token and written as
//              partial results per vocabulary split.
//   kGradient: with the per-token log-sum-exps known, the logit gradient
//              dO_S = coef_t (p_S - p_T), coef_t = grad_scale*m_t*lambda/tau (gradient of
//              Eq. 2), rounded to bf16 and stored to a scratch block that the two
//              backward contractions read.  With kComposite the cross-entropy term of
//              Eq. 1 is added: + cce_t (Softmax(O_S)[c] - [c = y_t]),
//              cce_t = grad_scale*m_t*(1-lambda).
//
// Two CTAs on neighbouring SMs (a cluster of 2) work as a pair on a 256-token x 256-column
// tile with tcgen05 .cta_group::2: each CTA stages its own 128 token rows of H and its own
// 128 of the tile's 256 weight rows, so a k-step costs each SM 32 KB of operand traffic
// instead of the 48 KB a lone 128 x 256 tile needs, and each CTA's tensor memory receives
// the logits of its own 128 tokens for all 256 columns.
//
// CTA = 384 threads, one CTA per SM, persistent over work units:
//   warp 0      TMA producer for this CTA's H and W operand stages (a ring of 3 stages of two k-steps in the
//               forward pass, of 5 single k-steps in the gradient pass); the
//               completion of both CTAs' loads is counted on the leader's "full" barrier
//   warp 1      leader CTA (cluster rank 0) only: tcgen05.mma issuer for the pair; commits
//               are multicast so that "stage free" and "accumulator ready" reach both CTAs.
//               In both CTAs this warp owns the 512 TMEM columns (2 accumulators 128x256).
//   warp 2      TMA producer for this CTA's teacher sub-tiles (a ring of 1 or 2 stages per column half); the rows of a
//               block lie anywhere in the packed batch, so each lane gathers four of them
//   warp 3      gradient pass only: one thread hands each finished gradient sub-tile to a TMA
//               store and recycles the stage when the store has read it
//   warps 4-11  epilogue; warp w reads TMEM lanes 32*(w%4).., columns 128*((w-4)/4)..
//               so every thread owns one token row and half of the tile's columns.
// The roles only ever meet at mbarriers (every wait on one is bounded), with one exception: with
// an fp32 teacher the four epilogue warps of a column half pass a named barrier before they
// overwrite the teacher sub-tile; that barrier carries a vote so that they leave together.
// All exponentials are taken in base 2 on logits pre-scaled by log2(e)/tau.
//
// kSparse: the teacher is given as its k largest logits per token (Eq. 2 as printed) instead
// of a dense row.  The forward then keeps the student's statistics only (the k teacher terms
// are evaluated per token afterwards), warp 2 has nothing to stream, and the gradient tile is
// coef_t p_S minus the k stored teacher probabilities at their columns.
//
// kTeacherF32: the dense teacher logits are fp32.  A sub-tile is then 128 rows x 32 columns
// (again 128-byte rows, 16 KB), read without unpacking; the bf16 gradient sub-tile (64-byte
// rows) no longer has the teacher's layout, so it is written unswizzled to the start of the
// stage once every thread of the half has its teacher values in registers.
#pragma once

#include "ptx_sm100.cuh"

namespace npd {

enum KdTileMode : int { kForward = 0, kGradient = 1 };

// Per-token fields of a forward partial (one partial per vocabulary split and column half).
enum : int { kPMaxA = 0, kPSumA, kPCross, kPMaxB, kPSumB, kPSumA1, kPSumB1, kPFields };

struct KdTileParams {
  int T, V;
  int ksteps;       // d / 64
  // The kernels work on the COMPACT rows: the tokens that carry loss, in packed order, numbered
  // 0..Tc-1 and cut into blocks of 128; a pair of CTAs owns two consecutive blocks.
  const int* plan;  // {blocks, pairs of blocks, forward runs, Tc}, written on the device
  const int* rows;  // [blocks*128] packed row (token) of every compact row; 0 beyond Tc
  int group_pairs;  // pairs of blocks per group: units are ordered group by group (within a group:
                    // pair fastest, then run), so that the H rows the CTA pairs work on at
                    // any one time stay in L2 while the W tiles are shared by a whole group
  int vt_begin;     // first 256-wide vocabulary tile of this launch
  int vt_count;     // number of vocabulary tiles of this launch; they are cut into runs (forward:
                    // plan[2] runs, gradient: one tile per run); a unit = (pair of blocks, run)
  float scale2;     // log2(e) / tau
  float tau;
  // forward
  float* partials;  // [2*nsplit][kPFields][T]
  int reverse;      // 1: the cross term is weighted by the student's probabilities (the divergence
                    // of the policy-lag monitor, student || given logits) instead of the teacher's
  // gradient
  // per-token arrays below are indexed by COMPACT row
  const float* lse2_a;  // [T] log2-sum-exp2 of the scaled teacher logits
  const float* lse2_b;  // [T] same for the student
  const float* coef;    // [T] grad_scale * m_t * lambda / tau
  // composite objective only (Eq. 1)
  const float* coef_ce;   // [T] grad_scale * m_t * [y_t >= 0] * (1 - lambda)
  const float* lse2_b1;   // [T] log2-sum-exp2 of the student logits * log2(e) (temperature 1)
  const int32_t* labels;  // [T], by token
  // top-k teacher only (kSparse)
  const int32_t* tk_idx;  // [T, topk] vocabulary indices of the stored teacher logits, by token
  const float* tk_cp;     // [T, topk] coef_t * p_T(j): what the gradient subtracts at column idx[t,j],
                          // by compact row
  int topk;               // <= kMaxTopK
  int g_col0;           // vocabulary column that scratch column 0 holds; scratch row = compact row
  int* status;
};

namespace kd_cfg {
constexpr int BM = 128, BN = 256, BK = 64, UK = 16;  // BM = token rows per CTA (256 per pair)
constexpr int BNH = BN / 2;                // weight rows each CTA of the pair stages
constexpr int A_BYTES = BM * BK * 2;       // 16 KB
constexpr int B_BYTES = BNH * BK * 2;      // 16 KB
constexpr int ZSUB_COLS = 64;              // teacher sub-tile: 128 rows x 64 bf16 (128 B rows)
constexpr int ZSUB_BYTES = BM * ZSUB_COLS * 2;  // 16 KB
constexpr int THREADS = 384;
constexpr int TMEM_COLS = 512;
// Shared-memory layout: 224 KB for the operand ring and the teacher stages (16 KB each, per
// column half).
// Every hand-off of an operand stage (the MMA issuer's wait for its loads, the release back to the
// TMA producer) costs the tensor pipe about 120 clocks whatever the stage holds, so the forward
// pass makes a stage two k-steps deep (64 KB, eight MMAs per hand-off instead of four): measured
// 10 % faster than single-k-step stages holding the same bytes.  Three such stages cover the latency
// of the loads; the 32 KB that remain give one teacher stage per half, which the forward epilogue
// tolerates (its warps hand a sub-tile back as soon as they have read it).  The gradient pass does
// not: its teacher stages double as staging for the gradient sub-tiles and are handed back only
// when the store of a sub-tile has read it, so it needs two of them per half and keeps five
// single-k-step operand stages (every variant with 64 KB stages was 9-24 % slower there).
template <int kMode>
struct Layout {
  static constexpr int KS = kMode == 0 ? 2 : 1;      // k-steps per operand stage
  static constexpr int STAGES = kMode == 0 ? 3 : 5;  // operand ring depth
  static constexpr int ZQ = kMode == 0 ? 1 : 2;      // teacher ring depth per column half
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = OFF_A + STAGES * KS * A_BYTES;
  static constexpr int OFF_Z = OFF_B + STAGES * KS * B_BYTES;
  static constexpr int OFF_BAR = OFF_Z + 2 * ZQ * ZSUB_BYTES;
  static constexpr int NUM_BARS = 2 * STAGES + 4 + 6 * ZQ;
  static constexpr int SMEM_BYTES = OFF_BAR + NUM_BARS * 8 + 16 + 1024;
};
// Teacher logits are clamped below at this value: a finite stand-in for the -inf entries of
// a densified top-k teacher.  It is small enough that 2^((clamp - row max) * scale) is 0 for
// any sane row, and small enough in magnitude that fp32 still resolves differences of scaled
// logits near it (a huge stand-in would turn "x*scale - max" into a rounding-error blow-up).
constexpr float kNegClamp = -30000.0f;
constexpr int kMaxTopK = 16;  // stored teacher logits per token the sparse path keeps in registers
}  // namespace kd_cfg

template <int kMode, bool kTauIsOne, bool kComposite, bool kSparse, bool kTeacherF32>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kd_cfg::THREADS, 1)
kd_tile_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_w,
               const __grid_constant__ CUtensorMap tmap_t, const __grid_constant__ CUtensorMap tmap_g,
               const KdTileParams p) {
  using namespace kd_cfg;
  using L = Layout<kMode>;
  constexpr int KS = L::KS, STAGES = L::STAGES, ZQ = L::ZQ, OFF_A = L::OFF_A, OFF_B = L::OFF_B, OFF_Z = L::OFF_Z,
                OFF_BAR = L::OFF_BAR, NUM_BARS = L::NUM_BARS;
  constexpr int ZC = kTeacherF32 ? 32 : ZSUB_COLS;  // columns of a teacher sub-tile (128-byte rows)
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + NUM_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();   // 0 = leader of the pair
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const uint32_t full0 = smem_u32(bars);
  const uint32_t empty0 = full0 + 8 * STAGES;
  const uint32_t tfull0 = empty0 + 8 * STAGES;
  const uint32_t tempty0 = tfull0 + 16;
  const uint32_t zfull0 = tempty0 + 16;           // [half][ZQ]
  const uint32_t zempty0 = zfull0 + 8 * 2 * ZQ;   // [half][ZQ]
  const uint32_t gfull0 = zempty0 + 8 * 2 * ZQ;   // [half][ZQ] gradient sub-tile written (gradient pass)

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull0 + 8 * b, 1);
      mbar_init(tempty0 + 8 * b, 16);  // 8 epilogue warps of each CTA, counted in the leader
    }
    for (int i = 0; i < 2 * ZQ; ++i) {
      mbar_init(zfull0 + 8 * i, 1);
      // a stage is given back by the four epilogue warps of its half (forward pass) or by the
      // thread that stores the gradient sub-tile once the store has read it (gradient pass)
      mbar_init(zempty0 + 8 * i, kMode == kForward ? 4 : 1);
      mbar_init(gfull0 + 8 * i, 4);
    }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_h);
    prefetch_tmap(&tmap_w);
    prefetch_tmap(&tmap_t);
    if (kMode == kGradient) prefetch_tmap(&tmap_g);
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything is sent to them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full_leader = mapa_shared(full0, 0);
  const uint32_t tempty_leader = mapa_shared(tempty0, 0);

  // Everything above touched only this CTA's own resources.  What follows reads what earlier
  // kernels in the stream wrote (the plan, the compact rows, the log-sum-exps) and overwrites
  // what they read (the gradient scratch), so it waits for them to be complete.
  grid_dependency_wait();
  grid_launch_dependents();

  const int nact = p.plan[0], pairs = p.plan[1];
  const int nsplit = kMode == kForward ? p.plan[2] : p.vt_count;
  const int units = pairs * nsplit;
  // slot = this CTA's block of compact rows, r = its first compact row, or -1 when the number of
  // blocks is odd and this CTA has none (it then stages block 0 and writes nothing).
  const int per_group = p.group_pairs * nsplit;  // units of a full group
  auto run_of = [&](int u, int& slot, int& r, int& s, int& vt0, int& vt1) {
    const int gi = u / per_group, local = u - gi * per_group;
    const int gsize = min(p.group_pairs, pairs - gi * p.group_pairs);
    s = local / gsize;
    slot = 2 * (gi * p.group_pairs + local % gsize) + static_cast<int>(rank);
    r = slot < nact ? slot * BM : -1;
    vt0 = p.vt_begin + static_cast<int>(static_cast<long long>(p.vt_count) * s / nsplit);
    vt1 = p.vt_begin + static_cast<int>(static_cast<long long>(p.vt_count) * (s + 1) / nsplit);
  };

  if (warp == 0) {
    // ---------------------- operand producer (H and W stages) ----------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int u = cluster_id; u < units && ok; u += num_clusters) {
        int slot, r, s, vt0, vt1;
        run_of(u, slot, r, s, vt0, vt1);
        const int rl = r < 0 ? 0 : r;
        for (int vt = vt0; vt < vt1 && ok; ++vt) {
          for (int ks = 0; ks < p.ksteps; ks += KS, ++it) {
            const uint32_t st = it % STAGES, ph = (it / STAGES) & 1;
            const int nk = min(KS, p.ksteps - ks);  // k-steps this stage carries
            if (!(ok = mbar_wait(empty0 + 8 * st, ph ^ 1, abort_flag))) break;
            // the leader's barrier counts the bytes of both CTAs' loads of this stage
            if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * st, 2 * nk * (A_BYTES + B_BYTES));
            const uint32_t fb = full_leader + 8 * st;
            for (int h = 0; h < nk; ++h) {
              tma_load_2d_pair(smem_u32(smem + OFF_A + (st * KS + h) * A_BYTES), &tmap_h, fb, (ks + h) * BK, rl);
              tma_load_2d_pair(smem_u32(smem + OFF_B + (st * KS + h) * B_BYTES), &tmap_w, fb, (ks + h) * BK,
                               vt * BN + static_cast<int>(rank) * BNH);
            }
          }
        }
      }
      // Drain: a stage is released only after its loads landed and the MMAs that read it
      // finished, so waiting for the release of the last stages covers both.
      const uint32_t last = it < STAGES ? it : STAGES;
      for (uint32_t j = 0; j < last && ok; ++j) {
        const uint32_t i2 = it - 1 - j;
        ok = mbar_wait(empty0 + 8 * (i2 % STAGES), (i2 / STAGES) & 1, abort_flag);
      }
      if (!ok) {
        // Aborted: nobody may be left to release the stages, but the loads already issued still
        // land in this CTA's shared memory.  The leader's "full" barriers count both CTAs' bytes;
        // the peer cannot wait on them and lets the grace period pass instead.
        if (rank == 0) {
          for (uint32_t j = 0; j < last; ++j) {
            const uint32_t i2 = it - 1 - j;
            mbar_wait_drain(full0 + 8 * (i2 % STAGES), (i2 / STAGES) & 1);
          }
        } else {
          grace_sleep();
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------- MMA issuer ----------------------
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * BM, BN, false, false);
      uint32_t it = 0, tile = 0;
      bool ok = true;
      for (int u = cluster_id; u < units && ok; u += num_clusters) {
        int slot, r, s, vt0, vt1;
        run_of(u, slot, r, s, vt0, vt1);
        (void)slot;
        for (int vt = vt0; vt < vt1 && ok; ++vt, ++tile) {
          const uint32_t buf = tile & 1, tph = (tile >> 1) & 1;
          if (!(ok = mbar_wait(tempty0 + 8 * buf, tph ^ 1, abort_flag))) break;
          tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + buf * BN;
          for (int ks = 0; ks < p.ksteps; ks += KS, ++it) {
            const uint32_t st = it % STAGES, ph = (it / STAGES) & 1;
            const int nk = min(KS, p.ksteps - ks);
            if (!(ok = mbar_wait(full0 + 8 * st, ph, abort_flag))) break;
            tc_fence_after_sync();
            for (int h = 0; h < nk; ++h) {
              const uint32_t sa = smem_u32(smem + OFF_A + (st * KS + h) * A_BYTES);
              const uint32_t sb = smem_u32(smem + OFF_B + (st * KS + h) * B_BYTES);
#pragma unroll
              for (int k = 0; k < BK / UK; ++k) {
                umma_bf16_pair(d_tmem, umma_desc_sw128(sa + k * (UK * 2), 16, 1024),
                               umma_desc_sw128(sb + k * (UK * 2), 16, 1024), idesc,
                               (ks > 0 || h > 0 || k > 0) ? 1u : 0u);
              }
            }
            umma_commit_pair(empty0 + 8 * st);
          }
          if (ok) umma_commit_pair(tfull0 + 8 * buf);
        }
      }
    }
  } else if (warp == 2) {
    // ---------------------- teacher producer ----------------------
    // The teacher rows of a block are scattered over the packed batch (the masked tokens in
    // between are left out), so a 128 x 64 sub-tile is fetched as 32 four-row gathers, one per
    // lane: lane l brings the block's rows 4l..4l+3 to their place in the swizzled sub-tile.
    if (!kSparse) {
      uint32_t zit = 0;  // sub-tile pairs issued; both halves advance together
      bool ok = true;
      for (int u = cluster_id; u < units && ok; u += num_clusters) {
        int slot, r, s, vt0, vt1;
        run_of(u, slot, r, s, vt0, vt1);
        int tr[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) tr[i] = r < 0 ? 0 : __ldg(p.rows + r + 4 * lane + i);
        for (int vt = vt0; vt < vt1 && ok; ++vt) {
          for (int j = 0; j < BN / 2 / ZC && ok; ++j, ++zit) {
            const uint32_t q = zit % ZQ, ph = (zit / ZQ) & 1;
            for (int half = 0; half < 2; ++half) {
              const int col = vt * BN + half * (BN / 2) + j * ZC;
              const uint32_t bi = 8 * (half * ZQ + q);
              ok = __all_sync(0xffffffffu, mbar_wait(zempty0 + bi, ph ^ 1, abort_flag));
              if (!ok) break;
              if (lane == 0) mbar_arrive_expect_tx(zfull0 + bi, ZSUB_BYTES);
              __syncwarp();
              tma_gather4_2d(smem_u32(smem + OFF_Z + (half * ZQ + q) * ZSUB_BYTES) + lane * 512, &tmap_t,
                             zfull0 + bi, col, tr[0], tr[1], tr[2], tr[3]);
            }
          }
        }
      }
      // Every gather issued must have landed before this CTA's shared memory is given up.  After
      // an abort the sub-tile pair that was being issued may be half out, so it is included; a
      // stage that was never armed just lets its (short) limit pass.
      const uint32_t upto = ok ? zit : zit + 1;
      const uint32_t last = upto < ZQ ? upto : ZQ;
      for (uint32_t j = 0; j < last; ++j) {
        const uint32_t i2 = upto - 1 - j;
        for (int half = 0; half < 2; ++half)
          mbar_wait_drain(zfull0 + 8 * (half * ZQ + (i2 % ZQ)), (i2 / ZQ) & 1);
      }
    }
  } else if (warp == 3) {
    // ---------------------- gradient sub-tile store (gradient pass) ----------------------
    // One thread hands every finished 128 x 64 gradient sub-tile to TMA and, once the store has
    // read it, gives the stage back (to the teacher producer, or with a top-k teacher to the
    // epilogue warps).  The epilogue warps never wait for a store.
    if (kMode == kGradient && lane == 0) {
      uint32_t zit = 0;
      bool ok = true;
      for (int u = cluster_id; u < units && ok; u += num_clusters) {
        int slot, r, s, vt0, vt1;
        run_of(u, slot, r, s, vt0, vt1);
        for (int vt = vt0; vt < vt1 && ok; ++vt) {
          for (int j = 0; j < BN / 2 / ZC && ok; ++j, ++zit) {
            const uint32_t q = zit % ZQ, ph = (zit / ZQ) & 1;
            for (int half = 0; half < 2 && ok; ++half) {
              const uint32_t bi = 8 * (half * ZQ + q);
              if (!(ok = mbar_wait(gfull0 + bi, ph, abort_flag))) break;
              if (r >= 0)
                tma_store_2d(&tmap_g, smem_u32(smem + OFF_Z + (half * ZQ + q) * ZSUB_BYTES),
                             vt * BN + half * (BN / 2) + j * ZC - p.g_col0, r);
            }
            if (!ok) break;
            tma_store_commit();
            tma_store_wait_read<0>();
            mbar_arrive(zempty0 + 8 * q);
            mbar_arrive(zempty0 + 8 * (ZQ + q));
          }
        }
      }
      tma_store_wait_all<0>();
    }
  } else if (warp >= 4) {
    // ---------------------- epilogue ----------------------
    const int e = warp - 4;
    const int lg = e & 3;      // == warp % 4: the TMEM lane group this warp may read
    const int half = e >> 2;   // which 128 columns of the 256-wide tile
    const int row_local = lg * 32 + lane;
    const uint32_t swz = static_cast<uint32_t>(row_local & 7);
    uint32_t tile = 0, zit = 0;
    bool ok = true;
    for (int u = cluster_id; u < units && ok; u += num_clusters) {
      int slot, r, s, vt0, vt1;
      run_of(u, slot, r, s, vt0, vt1);
      const int tc = p.plan[3];
      const int row = r < 0 ? tc : r + row_local;  // compact row; >= Tc: nothing to read or write
      // forward state (base-2 domain): running max / sum of the scaled teacher (a) and student (b)
      float m_a = -INFINITY, s_a = 0.f, cross = 0.f, m_b = -INFINITY, s_b = 0.f, s_a1 = 0.f, s_b1 = 0.f;
      // rows without a token (beyond T, or a CTA without a block): probabilities 0, gradient 0
      float g_lse_a = 1e30f, g_lse_b = 1e30f, g_coef = 0.f;
      float g_cce = 0.f, g_lse_b1 = 1e30f;  // cross-entropy term of the composite objective
      int g_y = -1;
      if (kMode == kGradient && row < tc) {
        g_lse_a = p.lse2_a[row];
        g_lse_b = p.lse2_b[row];
        g_coef = p.coef[row];
        if (kComposite) {
          g_cce = p.coef_ce[row];
          g_lse_b1 = p.lse2_b1[row];
          g_y = g_cce != 0.f ? p.labels[__ldg(p.rows + row)] : -1;
        }
      }
      // top-k teacher: this row's stored columns and what to subtract there
      int tki[kMaxTopK];
      float tkc[kMaxTopK];
      if (kSparse && kMode == kGradient) {
#pragma unroll
        for (int j = 0; j < kMaxTopK; ++j) {
          const bool have = row < tc && j < p.topk;
          tki[j] = have ? p.tk_idx[static_cast<size_t>(__ldg(p.rows + row)) * p.topk + j] : -1;
          tkc[j] = have ? p.tk_cp[static_cast<size_t>(row) * p.topk + j] : 0.f;
        }
      }
      for (int vt = vt0; vt < vt1 && ok; ++vt, ++tile) {
        const uint32_t buf = tile & 1, tph = (tile >> 1) & 1;
        // okw: this warp's waits so far succeeded.  A warp that gives up just leaves, except in the
        // gradient pass with an fp32 teacher: there the four warps of a column half meet at a
        // named barrier before they write, so a warp whose wait ran out still joins that barrier
        // (doing nothing else), and the barrier's vote tells the whole half to leave together.
        constexpr bool kMeets = kMode == kGradient && kTeacherF32;
        bool okw = __all_sync(0xffffffffu, mbar_wait(tfull0 + 8 * buf, tph, abort_flag));
        if (!kMeets && !okw) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t taddr =
            tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + buf * BN + half * (BN / 2);
        for (int j = 0; j < BN / 2 / ZC && ok; ++j, ++zit) {
          const uint32_t q = zit % ZQ, zph = (zit / ZQ) & 1;
          const uint32_t bi = 8 * (half * ZQ + q);
          if (!kSparse) {
            okw = okw && __all_sync(0xffffffffu, mbar_wait(zfull0 + bi, zph, abort_flag));
          } else if (kMode == kGradient) {
            // no teacher stream: the stage is free once the store of its last sub-tile has read it
            okw = okw && __all_sync(0xffffffffu, mbar_wait(zempty0 + bi, zph ^ 1, abort_flag));
          }
          if (!kMeets && !okw) { ok = false; break; }
          if (kMeets && !okw) {   // stands in for the barrier inside the loop below
            named_barrier_vote(1 + half, 128, false);
            ok = false;
            break;
          }
          uint8_t* zrow = smem + OFF_Z + (half * ZQ + q) * ZSUB_BYTES + row_local * 128;
          const int sub_col0 = vt * BN + half * (BN / 2) + j * ZC;
#pragma unroll 1
          for (int c = 0; okw && c < ZC / 32; ++c) {
            const int col0 = sub_col0 + c * 32;
            uint32_t acc[32];
            tmem_ld32(taddr + j * ZC + c * 32, acc);
            constexpr int NZQ = kTeacherF32 ? 8 : 4;  // 16-byte pieces that hold this chunk's 32 logits
            uint4 zq[NZQ];
            if (!kSparse) {
#pragma unroll
              for (int i = 0; i < NZQ; ++i)
                zq[i] = *reinterpret_cast<const uint4*>(
                    zrow + ((static_cast<uint32_t>(kTeacherF32 ? i : c * 4 + i) ^ swz) << 4));
            }
            tmem_ld_wait();
            const int nvalid = p.V - col0;  // columns of this chunk inside the vocabulary
            float zt[32];
            if (!kSparse) {
#pragma unroll
              for (int i = 0; i < NZQ; ++i) {
                const uint32_t w[4] = {zq[i].x, zq[i].y, zq[i].z, zq[i].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                  // (the gradient pass needs no clamp: 2^(-inf) is an exact zero there)
                  if (kTeacherF32) {
                    zt[4 * i + k] = kMode == kForward ? fmaxf(__uint_as_float(w[k]), kNegClamp) : __uint_as_float(w[k]);
                  } else {
                    zt[8 * i + 2 * k] = kMode == kForward ? fmaxf(bf16_lo(w[k]), kNegClamp) : bf16_lo(w[k]);
                    zt[8 * i + 2 * k + 1] = kMode == kForward ? fmaxf(bf16_hi(w[k]), kNegClamp) : bf16_hi(w[k]);
                  }
                }
              }
            }
            if (kMode == kForward && kSparse) {
              // student statistics only
              if (nvalid > 0) {
                float zs[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) zs[i] = (i < nvalid) ? __uint_as_float(acc[i]) : kNegClamp;
                float cb = zs[0];
#pragma unroll
                for (int i = 1; i < 32; ++i) cb = fmaxf(cb, zs[i]);
                cb *= p.scale2;
                if (cb > m_b) {
                  s_b *= ex2f(m_b - cb);
                  if (!kTauIsOne) s_b1 *= ex2f((m_b - cb) * p.tau);
                  m_b = cb;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                  const float tb = fmaf(zs[i], p.scale2, -m_b);
                  s_b += ex2f(tb);
                  if (!kTauIsOne) s_b1 += ex2f(tb * p.tau);
                }
              }
            } else if (kMode == kForward) {
              if (nvalid > 0) {
                float zs[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) zs[i] = __uint_as_float(acc[i]);
                if (nvalid < 32) {
#pragma unroll
                  for (int i = 0; i < 32; ++i)
                    if (i >= nvalid) { zs[i] = kNegClamp; zt[i] = kNegClamp; }
                }
                float ca = zt[0], cb = zs[0];
#pragma unroll
                for (int i = 1; i < 32; ++i) { ca = fmaxf(ca, zt[i]); cb = fmaxf(cb, zs[i]); }
                ca *= p.scale2;
                cb *= p.scale2;
                const bool rev = p.reverse != 0;  // uniform over the grid
                if (ca > m_a) {
                  const float f = ex2f(m_a - ca);
                  s_a *= f;
                  if (!rev) cross *= f;
                  if (!kTauIsOne) s_a1 *= ex2f((m_a - ca) * p.tau);
                  m_a = ca;
                }
                if (cb > m_b) {
                  const float f = ex2f(m_b - cb);
                  s_b *= f;
                  if (rev) cross *= f;
                  if (!kTauIsOne) s_b1 *= ex2f((m_b - cb) * p.tau);
                  m_b = cb;
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                  const float ta = fmaf(zt[i], p.scale2, -m_a);
                  const float tb = fmaf(zs[i], p.scale2, -m_b);
                  const float ea = ex2f(ta), eb = ex2f(tb);
                  s_a += ea;
                  cross = fmaf(rev ? eb : ea, zt[i] - zs[i], cross);
                  s_b += eb;
                  if (!kTauIsOne) {
                    s_a1 += ex2f(ta * p.tau);
                    s_b1 += ex2f(tb * p.tau);
                  }
                }
              }
            } else {
              // gradient tile: dO_S = coef * (p_S - p_T), written back in place over the teacher
              uint32_t packed[16];
              const int yi = kComposite ? g_y - col0 : -1;  // label's place in this chunk, if any
              float g[32];
#pragma unroll
              for (int i = 0; i < 32; ++i) {
                const float si = __uint_as_float(acc[i]);
                const float ps = ex2f(fmaf(si, p.scale2, -g_lse_b));
                g[i] = kSparse ? g_coef * ps : g_coef * (ps - ex2f(fmaf(zt[i], p.scale2, -g_lse_a)));
                if (kComposite) {
                  // at temperature 1 the two student softmaxes are the same
                  const float q = kTauIsOne ? ps : ex2f(fmaf(si, 1.4426950408889634f, -g_lse_b1));
                  g[i] = fmaf(g_cce, q - (i == yi ? 1.f : 0.f), g[i]);
                }
              }
              if (kSparse) {
                // the stored teacher probabilities that fall into this chunk (rare)
#pragma unroll
                for (int j = 0; j < kMaxTopK; ++j) {
                  const int dj = tki[j] - col0;
                  if (static_cast<unsigned>(dj) < 32u) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) g[i] -= (i == dj) ? tkc[j] : 0.f;
                  }
                }
              }
              if (nvalid >= 32) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) packed[i >> 1] = pack_bf16x2(g[i], g[i + 1]);
              } else {
#pragma unroll
                for (int i = 0; i < 32; i += 2)
                  packed[i >> 1] = pack_bf16x2(i < nvalid ? g[i] : 0.f, i + 1 < nvalid ? g[i + 1] : 0.f);
              }
              if (kTeacherF32) {
                // 64-byte gradient rows, dense from the start of the stage: they overlap other
                // threads' teacher rows, so everyone of this half must have read its row first
                if (!named_barrier_vote(1 + half, 128, true)) { ok = false; break; }
                uint8_t* grow = smem + OFF_Z + (half * ZQ + q) * ZSUB_BYTES + row_local * 64;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                  *reinterpret_cast<uint4*>(grow + 16 * i) =
                      make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
              } else {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                  *reinterpret_cast<uint4*>(zrow + ((static_cast<uint32_t>(c * 4 + i) ^ swz) << 4)) =
                      make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
              }
            }
          }
          if (kMode == kForward) {
            if (!kSparse) {
              __syncwarp();
              if (lane == 0) mbar_arrive(zempty0 + bi);
            }
          } else {
            // this warp's 32 rows of the gradient sub-tile are written: tell the storing thread
            if (!ok) break;
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(gfull0 + bi);
          }
        }
        if (!ok) break;
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);
      }
      if (kMode == kForward && ok && row < tc) {
        float* dst = p.partials + (static_cast<size_t>(2 * s + half) * kPFields) * p.T + row;
        dst[static_cast<size_t>(kPMaxA) * p.T] = m_a;
        dst[static_cast<size_t>(kPSumA) * p.T] = s_a;
        dst[static_cast<size_t>(kPCross) * p.T] = cross;
        dst[static_cast<size_t>(kPMaxB) * p.T] = m_b;
        dst[static_cast<size_t>(kPSumB) * p.T] = s_b;
        if (!kTauIsOne) {
          dst[static_cast<size_t>(kPSumA1) * p.T] = s_a1;
          dst[static_cast<size_t>(kPSumB1) * p.T] = s_b1;
        }
      }
    }
  }

  // ---------------------- teardown ----------------------
  // Neither CTA may leave (or free tensor memory) while its peer can still send it barrier
  // arrivals or have MMAs reading its shared memory.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && *abort_flag != 0 && p.status != nullptr) atomicCAS(p.status, 0, kStatusTimeout);
}

}  // namespace npd
