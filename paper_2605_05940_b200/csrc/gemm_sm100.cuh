// Persistent bf16 GEMM on tcgen05/TMEM with TMA-fed operands, used for the two
// backward contractions of the LM head (dH = dO_S W and dW = dO_S^T H, the
// chain rule through Algorithm 1's student-logit step).
//
//   D[M,N] (+)= sum_k A[m,k] * B[n,k]
//
// Either operand may be "K-major" (memory [rows][K contiguous]) or "MN-major"
// (memory [K][rows contiguous]); the second form lets the logit-gradient block
// and the hidden states be read as they lie in memory, with no transposes.
//
// One launch runs one or two such problems.  With two (the dW and dH products of one vocabulary
// chunk, which share N = d) the CTA pairs work in groups of as many pairs as a row tile has
// 512-wide column tiles: the members of a group take the column tiles of the SAME row tile at the
// same time, so the A operand they share (a panel of the logit-gradient block) is fetched from
// HBM once and served to the others from L2.  A group first takes whole row tiles of problem 0
// (last row tiles first: they are the part of the gradient block written last, still in L2);
// problem 1 is then laid out as one long line of (row tile, k-step) positions and every group gets
// the stretch of that line that brings it to the same total number of k-steps as all the others
// (a stretch may start and end in the middle of a tile: the pieces are added with fp32 atomics).
// Pairs that do not fill a group take whole tiles of problem 0 only.  This is how the two
// products share a launch and end together.
//
// Two CTAs on neighbouring SMs (a cluster of 2) work as a pair on a 256 x 512 output tile
// with tcgen05 .cta_group::2 (two M=256, N=256 accumulators that share the A operand): per
// k-step each CTA stages its own 128 rows of A and its own half (128 rows) of each of the two
// 256-row blocks of B, 48 KB for 2 x 128 x 256 x 64 MACs per SM.  This tile moves a quarter
// fewer operand bytes per MAC than a 256 x 256 pair tile (less power under the board's cap) and
// issues eight MMAs per k-step instead of four, which spreads the fixed cost of a k-step over
// twice the work; the price is that the 512 accumulator columns fill tensor memory, so the
// drain of a tile is not overlapped with the next tile's MMAs (a few per cent at the
// k-extents used here).
//
// One CTA per SM, 384 threads: warp 0 = TMA producer, warp 1 = TMEM owner and, in the leader
// CTA (cluster rank 0), the MMA issuer of the pair, warps 2-9 = epilogue in two groups of
// four warps (one accumulator row per thread, each group drains half of the columns), warps
// 10 and 11 = one storing thread per group.  An accumulator leaves through a ring of two small
// staging buffers per group: TMEM -> registers -> 64-byte-swizzled shared memory (128 rows x
// 64 bytes) -> TMA store, or TMA reduce-add for outputs that are accumulated (split-K, the
// stream-K pieces, several launches adding into one matrix).  The epilogue warps fill a buffer and
// signal it; the storing thread issues the copy and frees the buffer when the copy has read it,
// with one copy in flight while the next buffer is filled.  All roles meet at mbarriers only.
#pragma once

#include "ptx_sm100.cuh"

namespace npd {

struct GemmProblem {
  int M, N, K;
  int a_mn, b_mn;  // 1 = operand is MN-major
  int k_splits;    // > 1 only with out_reduce
  int out_f32;     // output elements: 1 = fp32, 0 = bf16
  int out_reduce;  // 1 = D += acc (atomic, any number of adders), 0 = D = acc
  // Extents only known on the device (the backward runs over the compact rows of a packed
  // batch, nblocks[0] blocks of 128):
  int dyn_m;       // M = 128 * nblocks[0]
  int dyn_k;       // K = 128 * nblocks[0]
  int stream_k;    // problem 1 only: cut along the (tile, k-step) line as described above
                   // (needs out_reduce and k_splits = 1)
};

struct GemmParams {
  GemmProblem pr[2];
  int nprob;           // 1 or 2
  const int* nblocks;  // device; read only when a problem has dyn_m / dyn_k
  int* status;         // device status word
};

namespace gemm_cfg {
constexpr int BM = 128;                 // rows per CTA
constexpr int PM = 2 * BM;              // rows of a pair tile
constexpr int BNS = 256;                // columns of one accumulator (the MMA's N)
constexpr int NSUB = 2;                 // accumulators per tile
constexpr int BN = BNS * NSUB;          // columns of a pair tile
constexpr int BK = 64, UK = 16, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;             // 16 KB
constexpr int BSUB_BYTES = (BNS / 2) * BK * 2;   // 16 KB: this CTA's half of one 256-row block of B
constexpr int B_BYTES = NSUB * BSUB_BYTES;       // 32 KB
constexpr int OUT_BYTES = 128 * 64;              // one staging buffer: 128 rows x 64 B
constexpr int OUT_BUFS = 2;                      // staging buffers per epilogue group
constexpr int THREADS = 384;
constexpr int TMEM_COLS = 512;
constexpr int OFF_A = 0;
constexpr int OFF_B = OFF_A + STAGES * A_BYTES;
constexpr int OFF_OUT = OFF_B + STAGES * B_BYTES;
constexpr int OFF_BAR = OFF_OUT + 2 * OUT_BUFS * OUT_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;  // + barriers + alignment
}  // namespace gemm_cfg

struct GemmUnit {
  int m0, n0, kt0, kt1;  // pair-tile origin and k-tile range
  int ns;                // accumulators in use: 2, or 1 when the tile's second 256 columns lie beyond N
};
// Tile `tile` (n fastest) of a problem, k-tiles [kt0, kt1).
__host__ __device__ __forceinline__ GemmUnit gemm_tile_unit(const GemmProblem& g, int tile, int kt0, int kt1) {
  using namespace gemm_cfg;
  const int tiles_n = (g.N + BN - 1) / BN;
  GemmUnit u;
  u.n0 = (tile % tiles_n) * BN;
  u.m0 = (tile / tiles_n) * PM;
  u.kt0 = kt0;
  u.kt1 = kt1;
  u.ns = (g.N - u.n0 > BNS) ? 2 : 1;
  return u;
}

// The sequence of units of one CTA pair.  Every role of both CTAs walks the same sequence.
struct GemmWalk {
  GemmProblem pr[2];
  int c, C;            // this pair and the number of pairs
  int tiles[2], ksteps[2];
  int i;               // units taken so far in the whole-tile phases
  long long pos, end;  // problem 1 with stream_k: this pair's stretch of the (tile, k-step) line
  // grouped mode (two problems that share N; see the head of this file)
  int grouped;
  int tn;              // column tiles per row tile = pairs per group
  int G;               // number of groups; pairs G*tn .. C-1 stand outside the groups
  int g, j;            // this pair's group and its column tile (g == G: outside the groups)
  int mt0, m_lone;     // row tiles of problem 0; the first m_lone of them go to the lone pairs
  int mine0;           // units of problem 0 this pair takes
  int lone_first;      // lone pair: its first tile (n fastest) of problem 0

  // nb = number of 128-row blocks behind the device-side extents (dyn_m / dyn_k)
  __host__ __device__ __forceinline__ void init(const GemmParams& p, int nb, int c_, int C_) {
    using namespace gemm_cfg;
    c = c_;
    C = C_;
    i = 0;
    pos = end = 0;
    grouped = 0;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      pr[q] = p.pr[q];
      if (pr[q].dyn_m) pr[q].M = 128 * nb;
      if (pr[q].dyn_k) pr[q].K = 128 * nb;
      tiles[q] = q < p.nprob ? ((pr[q].M + PM - 1) / PM) * ((pr[q].N + BN - 1) / BN) : 0;
      ksteps[q] = (pr[q].K + BK - 1) / BK;
    }
    tn = (pr[0].N + BN - 1) / BN;
    G = tn > 0 ? C / tn : 0;
    if (p.nprob == 2 && pr[1].stream_k && pr[0].k_splits == 1 && pr[0].N == pr[1].N && G > 0 &&
        tiles[0] > 0 && tiles[1] > 0 && ksteps[0] > 0 && ksteps[1] > 0) {
      grouped = 1;
      mt0 = tiles[0] / tn;
      const int mt1 = tiles[1] / tn;
      const int lone = C - G * tn;
      const double k0 = ksteps[0];
      const double line = static_cast<double>(mt1) * ksteps[1];
      // lone pairs: whole tiles of problem 0, no more than an even share of the launch's k-steps
      m_lone = 0;
      if (lone > 0) {
        const double share = (static_cast<double>(tiles[0]) * k0 + line * tn) / C;
        const int per = static_cast<int>(share / k0);
        m_lone = mt0 < lone * per / tn ? mt0 : lone * per / tn;
      }
      const int R = mt0 - m_lone;  // row tiles of problem 0 the groups take, round robin
      g = c / tn;
      j = c - g * tn;
      if (g >= G) {
        g = G;
        const int l = c - G * tn, xl = m_lone * tn, per = xl / lone, extra = xl % lone;
        lone_first = l * per + (l < extra ? l : extra);
        mine0 = per + (l < extra ? 1 : 0);
      } else {
        const int q0 = R / G, rem0 = R % G;
        mine0 = q0 + (g < rem0 ? 1 : 0);
        // groups 0..rem0-1 hold one more row tile of problem 0 and get the shorter stretch sa
        const double target = (R * k0 + line) / G;
        double sa = target - (q0 + 1) * k0;
        sa = sa > 0.0 ? sa : 0.0;
        const double sb = rem0 < G ? (line - rem0 * sa) / (G - rem0) : 0.0;
        auto prefix = [&](int k) { return k <= rem0 ? k * sa : rem0 * sa + (k - rem0) * sb; };
        pos = static_cast<long long>(prefix(g) + 0.5);
        end = g + 1 == G ? static_cast<long long>(line) : static_cast<long long>(prefix(g + 1) + 0.5);
      }
      return;
    }
    if (tiles[1] > 0 && pr[1].stream_k && ksteps[1] > 0) {
      // k-steps of problem 0 this pair and its neighbours carry (units go round robin)
      const int units0 = tiles[0] * pr[0].k_splits, q0 = units0 / C, rem0 = units0 % C;
      const double c0 = static_cast<double>((ksteps[0] + pr[0].k_splits - 1) / pr[0].k_splits);
      const double line = static_cast<double>(tiles[1]) * ksteps[1];
      const double target = (units0 * c0 + line) / C;
      // pairs 0..rem0-1 hold one more unit of problem 0 and get the shorter stretch sa
      double sa = target - (q0 + 1) * c0;
      sa = sa > 0.0 ? sa : 0.0;
      const double sb = rem0 < C ? (line - rem0 * sa) / (C - rem0) : 0.0;
      auto prefix = [&](int k) { return k <= rem0 ? k * sa : rem0 * sa + (k - rem0) * sb; };
      pos = static_cast<long long>(prefix(c) + 0.5);
      end = c + 1 == C ? static_cast<long long>(tiles[1]) * ksteps[1] : static_cast<long long>(prefix(c + 1) + 0.5);
    }
  }

  __host__ __device__ __forceinline__ bool next(int& prob, GemmUnit& u) {
    if (grouped) {
      if (i < mine0) {
        prob = 0;
        // lone pair: consecutive tiles; group member: its column tile of the group's i-th row tile,
        // the last row tiles first
        const int tile = g == G ? lone_first + i : (mt0 - 1 - (g + i * G)) * tn + j;
        u = gemm_tile_unit(pr[0], tile, 0, ksteps[0]);
        ++i;
        return true;
      }
      prob = 1;
      if (pos >= end) return false;
      const int m = static_cast<int>(pos / ksteps[1]), k0 = static_cast<int>(pos % ksteps[1]);
      const long long left = end - pos;
      const int len = left < ksteps[1] - k0 ? static_cast<int>(left) : ksteps[1] - k0;
      u = gemm_tile_unit(pr[1], m * tn + j, k0, k0 + len);
      pos += len;
      return true;
    }
    const int units0 = tiles[0] * pr[0].k_splits;
    const int mine = units0 / C + (c < units0 % C ? 1 : 0);
    if (i < mine) {
      const int v = c + i * C, ks = v / tiles[0];
      prob = 0;
      u = gemm_tile_unit(pr[0], v % tiles[0],
                         static_cast<int>(static_cast<long long>(ksteps[0]) * ks / pr[0].k_splits),
                         static_cast<int>(static_cast<long long>(ksteps[0]) * (ks + 1) / pr[0].k_splits));
      ++i;
      return true;
    }
    prob = 1;
    if (pr[1].stream_k) {
      if (pos >= end) return false;
      const int tile = static_cast<int>(pos / ksteps[1]), k0 = static_cast<int>(pos % ksteps[1]);
      const long long left = end - pos;
      const int len = left < ksteps[1] - k0 ? static_cast<int>(left) : ksteps[1] - k0;
      u = gemm_tile_unit(pr[1], tile, k0, k0 + len);
      pos += len;
      return true;
    }
    const int v = c + (i - mine) * C;
    if (v >= tiles[1] * pr[1].k_splits) return false;
    const int ks = v / tiles[1];
    u = gemm_tile_unit(pr[1], v % tiles[1],
                       static_cast<int>(static_cast<long long>(ksteps[1]) * ks / pr[1].k_splits),
                       static_cast<int>(static_cast<long long>(ksteps[1]) * (ks + 1) / pr[1].k_splits));
    ++i;
    return true;
  }
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(gemm_cfg::THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a0, const __grid_constant__ CUtensorMap tmap_b0,
                 const __grid_constant__ CUtensorMap tmap_o0, const __grid_constant__ CUtensorMap tmap_a1,
                 const __grid_constant__ CUtensorMap tmap_b1, const __grid_constant__ CUtensorMap tmap_o1,
                 const GemmParams p) {
  using namespace gemm_cfg;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* smem_a = smem + OFF_A;
  uint8_t* smem_b = smem + OFF_B;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  // bars[0..S) full, [S..2S) empty, [2S] tmem full, [2S+1] tmem empty,
  // [2S+2 ..) staging buffer filled [group][buffer], then staging buffer free [group][buffer]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2 + 4 * OUT_BUFS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);
  const uint32_t tfull = smem_u32(bars + 2 * STAGES), tempty = smem_u32(bars + 2 * STAGES + 1);
  const uint32_t ofull0 = smem_u32(bars + 2 * STAGES + 2), oempty0 = ofull0 + 8 * 2 * OUT_BUFS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    mbar_init(tfull, 1);
    mbar_init(tempty, 16);  // 8 epilogue warps of each CTA, counted in the leader
    for (int i = 0; i < 2 * OUT_BUFS; ++i) {
      mbar_init(ofull0 + 8 * i, 4);   // the four warps of the group
      mbar_init(oempty0 + 8 * i, 1);  // the group's storing thread
    }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_a0);
    prefetch_tmap(&tmap_b0);
    prefetch_tmap(&tmap_o0);
    if (p.nprob > 1) {
      prefetch_tmap(&tmap_a1);
      prefetch_tmap(&tmap_b1);
      prefetch_tmap(&tmap_o1);
    }
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything is sent to them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full_leader = mapa_shared(full0, 0);
  const uint32_t tempty_leader = mapa_shared(tempty, 0);

  // every role resolves the same problems and walks the same sequence of units
  // (the extents may come from the kernel before this one in the stream)
  grid_dependency_wait();
  grid_launch_dependents();
  GemmWalk walk;
  const bool dyn = p.pr[0].dyn_m || p.pr[0].dyn_k || p.pr[1].dyn_m || p.pr[1].dyn_k;
  walk.init(p, dyn ? __ldg(p.nblocks) : 0, cluster_id, num_clusters);

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      int prob;
      GemmUnit u;
      while (ok && walk.next(prob, u)) {
        const GemmProblem& g = prob ? walk.pr[1] : walk.pr[0];
        const CUtensorMap* ta = prob ? &tmap_a1 : &tmap_a0;
        const CUtensorMap* tb = prob ? &tmap_b1 : &tmap_b0;
        const int m0 = u.m0 + static_cast<int>(rank) * BM;          // this CTA's A rows
        const int n0 = u.n0 + static_cast<int>(rank) * (BNS / 2);   // its B rows within each 256-row block
        const uint32_t stage_bytes = 2 * (A_BYTES + u.ns * BSUB_BYTES);
        for (int kt = u.kt0; kt < u.kt1; ++kt, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!(ok = mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag))) break;
          // the leader's barrier counts the bytes of both CTAs' loads of this stage
          if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * s, stage_bytes);
          const uint32_t fb = full_leader + 8 * s;
          const uint32_t sa = smem_u32(smem_a + s * A_BYTES), sb = smem_u32(smem_b + s * B_BYTES);
          const int k0 = kt * BK;
          const int kb = k0;
          if (g.a_mn) {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d_pair(sa + j * 8192, ta, fb, m0 + 64 * j, k0);
          } else {
            tma_load_2d_pair(sa, ta, fb, k0, m0);
          }
          for (int h = 0; h < u.ns; ++h) {
            const uint32_t sbh = sb + h * BSUB_BYTES;
            const int nh = n0 + h * BNS;
            if (g.b_mn) {
#pragma unroll
              for (int j = 0; j < BNS / 2 / 64; ++j) tma_load_2d_pair(sbh + j * 8192, tb, fb, nh + 64 * j, kb);
            } else {
              tma_load_2d_pair(sbh, tb, fb, kb, nh);
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
    // ------------------------------ MMA issuer --------------------------------
    if (rank == 0 && lane == 0) {
      uint32_t it = 0, tile = 0;
      bool ok = true;
      int prob;
      GemmUnit u;
      for (; ok && walk.next(prob, u); ++tile) {
        const GemmProblem& g = prob ? walk.pr[1] : walk.pr[0];
        const uint32_t idesc = umma_idesc_bf16(PM, BNS, g.a_mn != 0, g.b_mn != 0);
        // the accumulators are free once every epilogue warp of the pair has read the last tile
        if (!(ok = mbar_wait(tempty, (tile & 1) ^ 1, abort_flag))) break;
        tc_fence_after_sync();
        // byte step between the four K=16 slices of a stage, and the descriptor's leading offset
        const uint32_t a_step = g.a_mn ? UK * 128 : UK * 2, a_lbo = g.a_mn ? BK * 128 : 16;
        const uint32_t b_step = g.b_mn ? UK * 128 : UK * 2, b_lbo = g.b_mn ? BK * 128 : 16;
        for (int kt = u.kt0; kt < u.kt1; ++kt, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!(ok = mbar_wait(full0 + 8 * s, ph, abort_flag))) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(smem_a + s * A_BYTES), sb = smem_u32(smem_b + s * B_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
            const uint64_t da = umma_desc_sw128(sa + k * a_step, a_lbo, 1024);
            const uint32_t acc = (kt > u.kt0 || k > 0) ? 1u : 0u;
            umma_bf16_pair(tmem_base, da, umma_desc_sw128(sb + k * b_step, b_lbo, 1024), idesc, acc);
            if (u.ns == 2)
              umma_bf16_pair(tmem_base + BNS, da, umma_desc_sw128(sb + BSUB_BYTES + k * b_step, b_lbo, 1024),
                             idesc, acc);
          }
          umma_commit_pair(empty0 + 8 * s);
        }
        if (ok) umma_commit_pair(tfull);
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------
    // What a group does with one unit, the same for its four warps and its storing thread:
    // sub-tiles of 64 output bytes per row (16 fp32 or 32 bf16 columns), `nsteps` of them.
    const bool storer = warp >= 10;
    const int grp = storer ? warp - 10 : (warp - 2) >> 2;  // which half of the tile's columns
    auto unit_steps = [&](const GemmProblem& g, const GemmUnit& u, int& c0, int& step) {
      const int gcols = (BNS / 2) * u.ns;         // accumulator columns this group drains
      c0 = grp * gcols;                           // the first of them
      step = g.out_f32 ? 16 : 32;
      const int m0 = u.m0 + static_cast<int>(rank) * BM;
      if (m0 >= g.M) return 0;                    // this CTA's 128 rows lie beyond M: nothing to store
      int n = (g.N - (u.n0 + c0) + step - 1) / step;  // sub-tiles of this group that lie inside N
      return n < 0 ? 0 : (n > gcols / step ? gcols / step : n);
    };
    uint32_t oit = 0;  // staging buffers used so far by this group (same count in all five roles)
    bool ok = true;
    int prob;
    GemmUnit u;
    if (storer) {
      if (lane == 0) {
        int prev = -1;  // buffer of the copy in flight
        while (ok && walk.next(prob, u)) {
          const GemmProblem& g = prob ? walk.pr[1] : walk.pr[0];
          const CUtensorMap* to = prob ? &tmap_o1 : &tmap_o0;
          int c0, step;
          const int nsteps = unit_steps(g, u, c0, step);
          const int row0 = u.m0 + static_cast<int>(rank) * BM;
          for (int j = 0; j < nsteps; ++j, ++oit) {
            const int b = grp * OUT_BUFS + static_cast<int>(oit % OUT_BUFS);
            if (!(ok = mbar_wait(ofull0 + 8 * b, (oit / OUT_BUFS) & 1, abort_flag))) break;
            const uint32_t src = smem_u32(smem + OFF_OUT + b * OUT_BYTES);
            const int col = u.n0 + c0 + j * step;
            if (g.out_reduce)
              tma_reduce_add_2d(to, src, col, row0);
            else
              tma_store_2d(to, src, col, row0);
            tma_store_commit();
            if (prev >= 0) {
              tma_store_wait_read<1>();  // the copy before this one has read its buffer
              mbar_arrive(oempty0 + 8 * prev);
            }
            prev = b;
          }
        }
        tma_store_wait_read<0>();
        if (prev >= 0) mbar_arrive(oempty0 + 8 * prev);
        tma_store_wait_all<0>();
      }
    } else {
      const int lg = warp & 3;   // TMEM lane group this warp may read
      const int row_local = lg * 32 + lane;
      const uint32_t swz = static_cast<uint32_t>((row_local >> 1) & 3);  // 64-byte swizzle
      uint32_t tile = 0;
      for (; ok && walk.next(prob, u); ++tile) {
        const GemmProblem& g = prob ? walk.pr[1] : walk.pr[0];
        const bool no_k = u.kt0 == u.kt1;           // empty k range: the accumulators hold nothing, D = 0
        int c0, step;
        const int nsteps = unit_steps(g, u, c0, step);
        ok = __all_sync(0xffffffffu, mbar_wait(tfull, tile & 1, abort_flag));
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + c0;
        if (nsteps == 0) {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tempty_leader);
        }
        for (int j = 0; j < nsteps; ++j, ++oit) {
          uint32_t w[16];  // 64 bytes of this thread's output row
          if (no_k) {
#pragma unroll
            for (int q = 0; q < 16; ++q) w[q] = 0u;
          } else if (g.out_f32) {
            tmem_ld16(taddr + j * 16, w);
            tmem_ld_wait();
          } else {
            uint32_t r0[32];
            tmem_ld32(taddr + j * 32, r0);
            tmem_ld_wait();
#pragma unroll
            for (int q = 0; q < 16; ++q)
              w[q] = pack_bf16x2(__uint_as_float(r0[2 * q]), __uint_as_float(r0[2 * q + 1]));
          }
          if (j == nsteps - 1) {
            // everything this warp needs from tensor memory is in registers: release the accumulators
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tempty_leader);
          }
          const int b = grp * OUT_BUFS + static_cast<int>(oit % OUT_BUFS);
          ok = __all_sync(0xffffffffu, mbar_wait(oempty0 + 8 * b, ((oit / OUT_BUFS) & 1) ^ 1, abort_flag));
          if (!ok) break;
          uint8_t* orow = smem + OFF_OUT + b * OUT_BYTES + row_local * 64;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4*>(orow + ((static_cast<uint32_t>(q) ^ swz) << 4)) =
                make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(ofull0 + 8 * b);
        }
      }
    }
  }

  // ------------------------------ teardown ------------------------------------
  // Neither CTA may leave (or free tensor memory) while its peer can still send it barrier
  // arrivals or have MMAs reading its shared memory.
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  tc_fence_after_sync();
  if (warp == 1) tmem_dealloc_pair(tmem_base, TMEM_COLS);
  if (threadIdx.x == 0 && *abort_flag != 0 && p.status != nullptr) atomicCAS(p.status, 0, kStatusTimeout);
}

}  // namespace npd
