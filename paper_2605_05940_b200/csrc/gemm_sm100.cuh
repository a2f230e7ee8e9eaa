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
// One launch runs one or two such problems.  With two, the CTA pairs first take the
// (long) units of problem 0 and then the (short, split-K) units of problem 1, dealt
// so that every pair ends at about the same time; this is how the dW and dH products
// of one vocabulary chunk share a launch without a tail in between.
//
// Two CTAs on neighbouring SMs (a cluster of 2) work as a pair on a 256 x 256 output tile
// with tcgen05 .cta_group::2: each CTA stages its own 128 rows of A and its own 128 of the
// tile's 256 rows of B (32 KB per k-step per SM) and receives its own 128 output rows in
// tensor memory.  One CTA per SM, 192 threads: warp 0 = TMA producer, warp 1 = TMEM owner
// and, in the leader CTA (cluster rank 0), the MMA issuer of the pair, warps 2-5 = epilogue
// (one accumulator row per thread).  6-stage operand ring, double-buffered accumulator
// (2 x 256 TMEM columns), so the epilogue of one unit overlaps the MMAs of the next.
#pragma once

#include "ptx_sm100.cuh"

namespace npd {

enum GemmOutMode : int {
  kOutStoreF32 = 0,   // D = acc
  kOutAddF32 = 1,     // D += acc (plain read-modify-write; each tile has one owner)
  kOutStoreBF16 = 2,  // D = bf16(acc)
  kOutAtomicF32 = 3,  // D += acc with red.global.add (split-K)
  kOutAddBF16 = 4     // D = bf16(D + acc)
};

struct GemmProblem {
  int M, N, K;
  int a_mn, b_mn;  // 1 = operand is MN-major
  int k_splits;    // > 1 only with kOutAtomicF32
  int out_mode;
  void* out;
  long long ldo;   // elements
};

struct GemmParams {
  GemmProblem pr[2];
  int units[2];    // work units of each problem (tiles x k_splits); units[1] = 0 for a single problem
  int q0, rem0;    // units[0] = q0 * pairs + rem0
  int extra1;      // units of problem 1 that each pair WITHOUT a remainder unit of problem 0 takes first
  int* status;     // device status word
};

namespace gemm_cfg {
constexpr int BM = 128, BN = 256, BK = 64, STAGES = 6, UK = 16;  // BM = rows per CTA (256 per pair)
constexpr int PM = 2 * BM;            // rows of a pair tile
constexpr int BNH = BN / 2;           // B rows each CTA of the pair stages
constexpr int A_BYTES = BM * BK * 2;  // 16 KB
constexpr int B_BYTES = BNH * BK * 2; // 16 KB
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int SMEM_BYTES = STAGES * (A_BYTES + B_BYTES) + 256 + 1024;  // + barriers + alignment
}  // namespace gemm_cfg

// The i-th unit of CTA pair c out of C.  Problem-0 units go round robin.  The pairs that got
// one unit fewer of problem 0 (c >= rem0) make up for it with `extra1` units of problem 1;
// the rest of problem 1 goes round robin over all pairs.
__host__ __device__ inline bool gemm_unit_at(const GemmParams& p, int c, int C, int i, int& prob, int& v) {
  const int n0 = p.q0 + (c < p.rem0 ? 1 : 0);
  if (i < n0) {
    prob = 0;
    v = c + i * C;
    return true;
  }
  prob = 1;
  int j = i - n0;
  int base = 0;
  if (p.rem0 > 0) {
    const int nb = C - p.rem0;
    base = p.extra1 * nb;
    if (c >= p.rem0) {
      if (j < p.extra1) {
        v = j * nb + (c - p.rem0);
        return v < p.units[1];
      }
      j -= p.extra1;
    }
  }
  v = base + j * C + c;
  return v < p.units[1];
}

struct GemmUnit {
  int m0, n0, kt0, kt1;  // pair-tile origin and k-tile range
};
__device__ __forceinline__ GemmUnit gemm_decode(const GemmProblem& g, int v) {
  using namespace gemm_cfg;
  const int tiles_m = (g.M + PM - 1) / PM, tiles_n = (g.N + BN - 1) / BN, ktiles = (g.K + BK - 1) / BK;
  const int ks = v / (tiles_n * tiles_m);
  GemmUnit u;
  u.n0 = (v % tiles_n) * BN;
  u.m0 = ((v / tiles_n) % tiles_m) * PM;
  u.kt0 = static_cast<int>(static_cast<long long>(ktiles) * ks / g.k_splits);
  u.kt1 = static_cast<int>(static_cast<long long>(ktiles) * (ks + 1) / g.k_splits);
  return u;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(gemm_cfg::THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a0, const __grid_constant__ CUtensorMap tmap_b0,
                 const __grid_constant__ CUtensorMap tmap_a1, const __grid_constant__ CUtensorMap tmap_b1,
                 const GemmParams p) {
  using namespace gemm_cfg;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_BYTES + B_BYTES));
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem full, [2S+2..2S+4) tmem empty
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const int cluster_id = blockIdx.x >> 1;
  const int num_clusters = gridDim.x >> 1;
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);
  const uint32_t tfull0 = smem_u32(bars + 2 * STAGES), tempty0 = smem_u32(bars + 2 * STAGES + 2);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full0 + 8 * s, 1);
      mbar_init(empty0 + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull0 + 8 * b, 1);
      mbar_init(tempty0 + 8 * b, 8);  // 4 epilogue warps of each CTA, counted in the leader
    }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmap_a0);
    prefetch_tmap(&tmap_b0);
    if (p.units[1] > 0) {
      prefetch_tmap(&tmap_a1);
      prefetch_tmap(&tmap_b1);
    }
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything is sent to them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full_leader = mapa_shared(full0, 0);
  const uint32_t tempty_leader = mapa_shared(tempty0, 0);

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      int prob, v;
      for (int i = 0; ok && gemm_unit_at(p, cluster_id, num_clusters, i, prob, v); ++i) {
        const GemmProblem& g = p.pr[prob];
        const GemmUnit u = gemm_decode(g, v);
        const CUtensorMap* ta = prob ? &tmap_a1 : &tmap_a0;
        const CUtensorMap* tb = prob ? &tmap_b1 : &tmap_b0;
        const int m0 = u.m0 + static_cast<int>(rank) * BM;   // this CTA's A rows
        const int n0 = u.n0 + static_cast<int>(rank) * BNH;  // and B rows
        for (int kt = u.kt0; kt < u.kt1; ++kt, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!(ok = mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag))) break;
          // the leader's barrier counts the bytes of both CTAs' loads of this stage
          if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * s, 2 * (A_BYTES + B_BYTES));
          const uint32_t fb = full_leader + 8 * s;
          const uint32_t sa = smem_u32(smem_a + s * A_BYTES), sb = smem_u32(smem_b + s * B_BYTES);
          const int k0 = kt * BK;
          if (g.a_mn) {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d_pair(sa + j * 8192, ta, fb, m0 + 64 * j, k0);
          } else {
            tma_load_2d_pair(sa, ta, fb, k0, m0);
          }
          if (g.b_mn) {
#pragma unroll
            for (int j = 0; j < BNH / 64; ++j) tma_load_2d_pair(sb + j * 8192, tb, fb, n0 + 64 * j, k0);
          } else {
            tma_load_2d_pair(sb, tb, fb, k0, n0);
          }
        }
      }
      // Drain: a stage is released only after its loads landed and the MMAs that read it
      // finished, so waiting for the release of the last stages covers both.
      const uint32_t last = it < STAGES ? it : STAGES;
      for (uint32_t j = 0; j < last; ++j) {
        const uint32_t i2 = it - 1 - j;
        mbar_wait(empty0 + 8 * (i2 % STAGES), (i2 / STAGES) & 1, abort_flag);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    if (rank == 0 && lane == 0) {
      uint32_t it = 0, tile = 0;
      bool ok = true;
      int prob, v;
      for (int i = 0; ok && gemm_unit_at(p, cluster_id, num_clusters, i, prob, v); ++i, ++tile) {
        const GemmProblem& g = p.pr[prob];
        const GemmUnit u = gemm_decode(g, v);
        const uint32_t idesc = umma_idesc_bf16(PM, BN, g.a_mn != 0, g.b_mn != 0);
        const uint32_t buf = tile & 1, tph = (tile >> 1) & 1;
        if (!(ok = mbar_wait(tempty0 + 8 * buf, tph ^ 1, abort_flag))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + buf * BN;
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
            umma_bf16_pair(d_tmem, umma_desc_sw128(sa + k * a_step, a_lbo, 1024),
                           umma_desc_sw128(sb + k * b_step, b_lbo, 1024), idesc,
                           (kt > u.kt0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(empty0 + 8 * s);
        }
        if (ok) umma_commit_pair(tfull0 + 8 * buf);
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------
    const int lg = warp & 3;  // TMEM lane group this warp may read
    uint32_t tile = 0;
    bool ok = true;
    int prob, v;
    for (int i = 0; ok && gemm_unit_at(p, cluster_id, num_clusters, i, prob, v); ++i, ++tile) {
      const GemmProblem& g = p.pr[prob];
      const GemmUnit u = gemm_decode(g, v);
      const int n0 = u.n0;
      const int m0 = u.m0 + static_cast<int>(rank) * BM;
      const int out_mode = g.out_mode;
      const uint32_t buf = tile & 1, tph = (tile >> 1) & 1;
      if (!(ok = mbar_wait(tfull0 + 8 * buf, tph, abort_flag))) break;
      tc_fence_after_sync();
      const int row = m0 + lg * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + buf * BN;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        const int col0 = n0 + c * 32;
        if (col0 >= g.N) break;  // uniform over the warp
        uint32_t r[32];
        tmem_ld32(taddr + c * 32, r);
        tmem_ld_wait();
        if (row < g.M) {
          const bool full_chunk = (col0 + 32 <= g.N);
          if (out_mode == kOutStoreBF16 || out_mode == kOutAddBF16) {
            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(g.out) + row * g.ldo + col0;
            if (full_chunk) {
              uint4* o4 = reinterpret_cast<uint4*>(o);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                float x[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) x[q] = __uint_as_float(r[8 * j + q]);
                if (out_mode == kOutAddBF16) {
                  const uint4 old = o4[j];
                  x[0] += bf16_lo(old.x); x[1] += bf16_hi(old.x);
                  x[2] += bf16_lo(old.y); x[3] += bf16_hi(old.y);
                  x[4] += bf16_lo(old.z); x[5] += bf16_hi(old.z);
                  x[6] += bf16_lo(old.w); x[7] += bf16_hi(old.w);
                }
                uint4 w;
                w.x = pack_bf16x2(x[0], x[1]);
                w.y = pack_bf16x2(x[2], x[3]);
                w.z = pack_bf16x2(x[4], x[5]);
                w.w = pack_bf16x2(x[6], x[7]);
                o4[j] = w;
              }
            } else {
              for (int j = 0; j < 32 && col0 + j < g.N; ++j) {
                float x = __uint_as_float(r[j]);
                if (out_mode == kOutAddBF16) x += __bfloat162float(o[j]);
                o[j] = __float2bfloat16_rn(x);
              }
            }
          } else {
            float* o = reinterpret_cast<float*>(g.out) + row * g.ldo + col0;
            if (out_mode == kOutAtomicF32) {
              if (full_chunk) {
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(o + j),
                               "f"(__uint_as_float(r[j])), "f"(__uint_as_float(r[j + 1])),
                               "f"(__uint_as_float(r[j + 2])), "f"(__uint_as_float(r[j + 3]))
                               : "memory");
              } else {
                for (int j = 0; j < 32 && col0 + j < g.N; ++j) atomicAdd(o + j, __uint_as_float(r[j]));
              }
            } else if (full_chunk) {
              float4* o4 = reinterpret_cast<float4*>(o);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float4 x = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                       __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                if (out_mode == kOutAddF32) {
                  const float4 old = o4[j];
                  x.x += old.x; x.y += old.y; x.z += old.z; x.w += old.w;
                }
                o4[j] = x;
              }
            } else {
              for (int j = 0; j < 32 && col0 + j < g.N; ++j) {
                float x = __uint_as_float(r[j]);
                if (out_mode == kOutAddF32) x += o[j];
                o[j] = x;
              }
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);
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
