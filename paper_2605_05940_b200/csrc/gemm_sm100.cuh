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
// Two CTAs on neighbouring SMs (a cluster of 2) work as a pair on a 256 x 256 output tile
// with tcgen05 .cta_group::2: each CTA stages its own 128 rows of A and its own 128 of the
// tile's 256 rows of B (32 KB per k-step per SM) and receives its own 128 output rows in
// tensor memory.  One CTA per SM, 192 threads: warp 0 = TMA producer, warp 1 = TMEM owner
// and, in the leader CTA (cluster rank 0), the MMA issuer of the pair, warps 2-5 = epilogue
// (one accumulator row per thread).  6-stage operand ring, double-buffered accumulator
// (2 x 256 TMEM columns), so the epilogue of one tile overlaps the MMAs of the next.
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

struct GemmParams {
  int M, N, K;
  int k_splits;   // > 1 only with kOutAtomicF32
  void* out;
  long long ldo;  // elements
  int out_mode;
  int* status;    // device status word
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

template <bool kAMn, bool kBMn>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(gemm_cfg::THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
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
    prefetch_tmap(&tmap_a);
    prefetch_tmap(&tmap_b);
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything is sent to them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full_leader = mapa_shared(full0, 0);
  const uint32_t tempty_leader = mapa_shared(tempty0, 0);

  const int tiles_m = (p.M + PM - 1) / PM;
  const int tiles_n = (p.N + BN - 1) / BN;
  const int ktiles = (p.K + BK - 1) / BK;
  const int units = tiles_m * tiles_n * p.k_splits;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int u = cluster_id; u < units && ok; u += num_clusters) {
        const int n0 = (u % tiles_n) * BN + static_cast<int>(rank) * BNH;        // this CTA's B rows
        const int m0 = ((u / tiles_n) % tiles_m) * PM + static_cast<int>(rank) * BM;  // and A rows
        const int ks = u / (tiles_n * tiles_m);
        const int kt0 = static_cast<int>(static_cast<long long>(ktiles) * ks / p.k_splits);
        const int kt1 = static_cast<int>(static_cast<long long>(ktiles) * (ks + 1) / p.k_splits);
        for (int kt = kt0; kt < kt1; ++kt, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!(ok = mbar_wait(empty0 + 8 * s, ph ^ 1, abort_flag))) break;
          // the leader's barrier counts the bytes of both CTAs' loads of this stage
          if (rank == 0) mbar_arrive_expect_tx(full0 + 8 * s, 2 * (A_BYTES + B_BYTES));
          const uint32_t fb = full_leader + 8 * s;
          const uint32_t sa = smem_u32(smem_a + s * A_BYTES), sb = smem_u32(smem_b + s * B_BYTES);
          const int k0 = kt * BK;
          if (kAMn) {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) tma_load_2d_pair(sa + i * 8192, &tmap_a, fb, m0 + 64 * i, k0);
          } else {
            tma_load_2d_pair(sa, &tmap_a, fb, k0, m0);
          }
          if (kBMn) {
#pragma unroll
            for (int i = 0; i < BNH / 64; ++i) tma_load_2d_pair(sb + i * 8192, &tmap_b, fb, n0 + 64 * i, k0);
          } else {
            tma_load_2d_pair(sb, &tmap_b, fb, k0, n0);
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
      constexpr uint32_t idesc = umma_idesc_bf16(PM, BN, kAMn, kBMn);
      uint32_t it = 0, tile = 0;
      bool ok = true;
      for (int u = cluster_id; u < units && ok; u += num_clusters, ++tile) {
        const int ks = u / (tiles_n * tiles_m);
        const int kt0 = static_cast<int>(static_cast<long long>(ktiles) * ks / p.k_splits);
        const int kt1 = static_cast<int>(static_cast<long long>(ktiles) * (ks + 1) / p.k_splits);
        const uint32_t buf = tile & 1, tph = (tile >> 1) & 1;
        if (!(ok = mbar_wait(tempty0 + 8 * buf, tph ^ 1, abort_flag))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kt = kt0; kt < kt1; ++kt, ++it) {
          const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
          if (!(ok = mbar_wait(full0 + 8 * s, ph, abort_flag))) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(smem_a + s * A_BYTES), sb = smem_u32(smem_b + s * B_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UK; ++k) {
            const uint64_t da = kAMn ? umma_desc_sw128(sa + k * (UK * 128), BK * 128, 1024)
                                     : umma_desc_sw128(sa + k * (UK * 2), 16, 1024);
            const uint64_t db = kBMn ? umma_desc_sw128(sb + k * (UK * 128), BK * 128, 1024)
                                     : umma_desc_sw128(sb + k * (UK * 2), 16, 1024);
            umma_bf16_pair(d_tmem, da, db, idesc, (kt > kt0 || k > 0) ? 1u : 0u);
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
    for (int u = cluster_id; u < units && ok; u += num_clusters, ++tile) {
      const int n0 = (u % tiles_n) * BN;
      const int m0 = ((u / tiles_n) % tiles_m) * PM + static_cast<int>(rank) * BM;
      const uint32_t buf = tile & 1, tph = (tile >> 1) & 1;
      if (!(ok = mbar_wait(tfull0 + 8 * buf, tph, abort_flag))) break;
      tc_fence_after_sync();
      const int row = m0 + lg * 32 + lane;
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16) + buf * BN;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(taddr + c * 32, r);
        tmem_ld_wait();
        const int col0 = n0 + c * 32;
        if (row < p.M && col0 < p.N) {
          const bool full_chunk = (col0 + 32 <= p.N);
          if (p.out_mode == kOutStoreBF16 || p.out_mode == kOutAddBF16) {
            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + row * p.ldo + col0;
            if (full_chunk) {
              uint4* o4 = reinterpret_cast<uint4*>(o);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                float v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = __uint_as_float(r[8 * j + q]);
                if (p.out_mode == kOutAddBF16) {
                  const uint4 old = o4[j];
                  v[0] += bf16_lo(old.x); v[1] += bf16_hi(old.x);
                  v[2] += bf16_lo(old.y); v[3] += bf16_hi(old.y);
                  v[4] += bf16_lo(old.z); v[5] += bf16_hi(old.z);
                  v[6] += bf16_lo(old.w); v[7] += bf16_hi(old.w);
                }
                uint4 w;
                w.x = pack_bf16x2(v[0], v[1]);
                w.y = pack_bf16x2(v[2], v[3]);
                w.z = pack_bf16x2(v[4], v[5]);
                w.w = pack_bf16x2(v[6], v[7]);
                o4[j] = w;
              }
            } else {
              for (int j = 0; j < 32 && col0 + j < p.N; ++j) {
                float v = __uint_as_float(r[j]);
                if (p.out_mode == kOutAddBF16) v += __bfloat162float(o[j]);
                o[j] = __float2bfloat16_rn(v);
              }
            }
          } else {
            float* o = reinterpret_cast<float*>(p.out) + row * p.ldo + col0;
            if (p.out_mode == kOutAtomicF32) {
              if (full_chunk) {
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(o + j),
                               "f"(__uint_as_float(r[j])), "f"(__uint_as_float(r[j + 1])),
                               "f"(__uint_as_float(r[j + 2])), "f"(__uint_as_float(r[j + 3]))
                               : "memory");
              } else {
                for (int j = 0; j < 32 && col0 + j < p.N; ++j) atomicAdd(o + j, __uint_as_float(r[j]));
              }
            } else if (full_chunk) {
              float4* o4 = reinterpret_cast<float4*>(o);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                       __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                if (p.out_mode == kOutAddF32) {
                  const float4 old = o4[j];
                  v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
                }
                o4[j] = v;
              }
            } else {
              for (int j = 0; j < 32 && col0 + j < p.N; ++j) {
                float v = __uint_as_float(r[j]);
                if (p.out_mode == kOutAddF32) v += o[j];
                o[j] = v;
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
