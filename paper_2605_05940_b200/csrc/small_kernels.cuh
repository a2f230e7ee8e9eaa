// The per-token and per-sample kernels around the tensor-core tiles: merging the
// forward partials into losses, segment reductions over cu_seqlens, the Delta-IFD
// score and selection, and a few layout helpers.  All fp32, deterministic.
#pragma once

#include "kd_tile_sm100.cuh"

namespace npd {

constexpr float kLn2 = 0.693147180559945309417f;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Rounds-times-tiles cost of cutting `vtiles` vocabulary tiles into ns runs for `pairs` row
// pairs on `clusters` CTA pairs; the smallest cost wins (ties: fewer runs).
__host__ __device__ inline int choose_nsplit(int pairs, int vtiles, int clusters, int nsplit_max) {
  int best = 1;
  long long best_cost = -1;
  for (int ns = 1; ns <= nsplit_max && ns <= vtiles; ++ns) {
    const long long rounds = (static_cast<long long>(pairs) * ns + clusters - 1) / clusters;
    const long long per = (vtiles + ns - 1) / ns;
    const long long cost = rounds * per * 64 + ns;
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = ns;
    }
  }
  return best;
}

// One CTA.  Numbers the tokens that carry loss (m_t = 1) in packed order: compact row c of
// token t = the count of loss tokens before t.  Tokens without loss have zero loss and zero
// gradient, and no tile of any later kernel is spent on them: the tile kernels and the
// contractions run over the compact rows 0..Tc-1, cut into blocks of 128.
//   rows[c] = token of compact row c (0 for the padding rows Tc .. blocks*128-1)
//   cidx[t] = compact row of token t, or -1
//   plan    = {blocks, pairs of blocks, forward runs, Tc}
__global__ void __launch_bounds__(1024) plan_rows_kernel(int T, const uint8_t* __restrict__ mask,
                                                         int vtiles, int nsplit_max, int clusters,
                                                         int* plan, int* rows, int* cidx) {
  __shared__ int warp_tot[32];
  __shared__ int total;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int per = (T + 1023) / 1024;                 // consecutive tokens per thread
  const int t0 = min(T, static_cast<int>(threadIdx.x) * per), t1 = min(T, t0 + per);
  int cnt = 0;
  for (int t = t0; t < t1; ++t) cnt += (mask == nullptr || mask[t] != 0) ? 1 : 0;
  // exclusive scan of cnt over the CTA
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_tot[lane], wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += v;
    }
    warp_tot[lane] = wi - w;                          // exclusive offsets of the warps
    if (lane == 31) total = wi;
  }
  __syncthreads();
  int c = warp_tot[warp] + incl - cnt;
  for (int t = t0; t < t1; ++t) {
    const bool on = mask == nullptr || mask[t] != 0;
    cidx[t] = on ? c : -1;
    if (on) rows[c++] = t;
  }
  const int tc = total, nact = (tc + 127) / 128, pairs = (nact + 1) / 2;
  for (int i = tc + threadIdx.x; i < nact * 128; i += blockDim.x) rows[i] = 0;
  if (threadIdx.x == 0) {
    plan[0] = nact;
    plan[1] = pairs;
    plan[2] = choose_nsplit(pairs > 0 ? pairs : 1, vtiles, clusters, nsplit_max);
    plan[3] = tc;
  }
}

// Copies the hidden states of the compact rows next to each other (the padding rows of the last
// block become zeros), so that the tile kernels and the dW contraction read them with plain
// tiled TMA loads.  8 elements per thread.
__global__ void __launch_bounds__(256) gather_hidden_rows_kernel(const __nv_bfloat16* __restrict__ H,
                                                                 long long ldh, int d,
                                                                 const int* __restrict__ plan,
                                                                 const int* __restrict__ rows,
                                                                 __nv_bfloat16* Hc) {
  const int per_row = d / 8;
  const long long n = static_cast<long long>(plan[0]) * 128 * per_row;
  for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int c = static_cast<int>(i / per_row), k = static_cast<int>(i % per_row) * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (c < plan[3]) v = *reinterpret_cast<const uint4*>(H + static_cast<size_t>(rows[c]) * ldh + k);
    *reinterpret_cast<uint4*>(Hc + static_cast<size_t>(c) * d + k) = v;
  }
}

struct CombineParams {
  int T, d, V;
  const int* plan;        // plan[2] = forward runs; the partials hold 2 slots per run
  const int* cidx;        // [T] compact row of a token (partials, lse2_*, coef* are indexed by it)
  const float* partials;  // [nslots][kPFields][T]
  const __nv_bfloat16* hidden;
  const __nv_bfloat16* weight;
  const void* teacher;    // bf16, or fp32 when teacher_f32
  int teacher_f32;
  long long ldh, ldw, ldt;
  const uint8_t* loss_mask;
  const int32_t* labels;
  float scale2, tau, grad_scale;
  float* kl;
  float* nll_s;
  float* nll_t;
  float* lse2_a;
  float* lse2_b;
  float* coef;
  // composite objective (Eq. 1): lambda weighs the distillation term, 1 - lambda the
  // cross-entropy; coef_ce / lse2_b1 are NULL when the objective is Eq. 2 alone (lambda = 1)
  float lambda;
  float* coef_ce;
  float* lse2_b1;
  int reverse;  // 1: kl[t] = D(student || given logits), the cross partials carry the student's weights
};

// One warp per token.  Merges the per-split online-softmax partials into the token's
// log-sum-exps, evaluates Eq. 2 as  KL = sum_c p_T(c)(a_c - b_c) - lse(a) + lse(b)
// (a, b the temperature-scaled teacher / student logits) and the two label
// cross-entropies behind Eq. 3, and saves what the gradient tiles need.
template <bool kTauIsOne>
__global__ void __launch_bounds__(256) kd_combine_kernel(const CombineParams p) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= p.T) return;
  const size_t fs = static_cast<size_t>(p.T);            // field stride
  const size_t ss = static_cast<size_t>(kPFields) * fs;  // slot stride
  const int nslots = 2 * p.plan[2];
  const bool on = p.loss_mask == nullptr || p.loss_mask[t] != 0;
  if (!on) {
    // no loss and no gradient here, and no compact row: nothing was computed for this token
    if (lane == 0) {
      p.kl[t] = 0.f;
      if (p.nll_s != nullptr) p.nll_s[t] = 0.f;
      if (p.nll_t != nullptr) p.nll_t[t] = 0.f;
    }
    return;
  }
  const int c = p.cidx[t];  // the token's compact row
  float ma = -INFINITY, mb = -INFINITY;
  for (int s = lane; s < nslots; s += 32) {
    const float* q = p.partials + s * ss + c;
    ma = fmaxf(ma, q[kPMaxA * fs]);
    mb = fmaxf(mb, q[kPMaxB * fs]);
  }
  ma = warp_max(ma);
  mb = warp_max(mb);
  float sa = 0.f, cr = 0.f, sb = 0.f, sa1 = 0.f, sb1 = 0.f;
  for (int s = lane; s < nslots; s += 32) {
    const float* q = p.partials + s * ss + c;
    const float da = q[kPMaxA * fs] - ma, db = q[kPMaxB * fs] - mb;
    const float fa = exp2f(da), fb = exp2f(db);
    sa = fmaf(q[kPSumA * fs], fa, sa);
    cr = fmaf(q[kPCross * fs], p.reverse ? fb : fa, cr);
    sb = fmaf(q[kPSumB * fs], fb, sb);
    if (!kTauIsOne) {
      sa1 = fmaf(q[kPSumA1 * fs], exp2f(da * p.tau), sa1);
      sb1 = fmaf(q[kPSumB1 * fs], exp2f(db * p.tau), sb1);
    }
  }
  sa = warp_sum(sa);
  cr = warp_sum(cr);
  sb = warp_sum(sb);
  if (!kTauIsOne) {
    sa1 = warp_sum(sa1);
    sb1 = warp_sum(sb1);
  }
  const float lse_a = ma + log2f(sa), lse_b = mb + log2f(sb);

  // label logits: O_S[t, y] = <H[t], W[y]> in fp32, O_T[t, y] read directly
  float nll_s = 0.f, nll_t = 0.f;
  bool has_label = false;
  if (p.labels != nullptr) {
    const int y = p.labels[t];
    if (on && y >= 0 && y < p.V) {
      has_label = true;
      const uint4* h4 = reinterpret_cast<const uint4*>(p.hidden + static_cast<size_t>(t) * p.ldh);
      const uint4* w4 = reinterpret_cast<const uint4*>(p.weight + static_cast<size_t>(y) * p.ldw);
      float dot = 0.f;
      for (int i = lane; i < p.d / 8; i += 32) {
        const uint4 h = h4[i], w = w4[i];
        dot = fmaf(bf16_lo(h.x), bf16_lo(w.x), dot);
        dot = fmaf(bf16_hi(h.x), bf16_hi(w.x), dot);
        dot = fmaf(bf16_lo(h.y), bf16_lo(w.y), dot);
        dot = fmaf(bf16_hi(h.y), bf16_hi(w.y), dot);
        dot = fmaf(bf16_lo(h.z), bf16_lo(w.z), dot);
        dot = fmaf(bf16_hi(h.z), bf16_hi(w.z), dot);
        dot = fmaf(bf16_lo(h.w), bf16_lo(w.w), dot);
        dot = fmaf(bf16_hi(h.w), bf16_hi(w.w), dot);
      }
      dot = warp_sum(dot);
      const size_t at = static_cast<size_t>(t) * p.ldt + y;
      const float zt_y = p.teacher_f32 ? static_cast<const float*>(p.teacher)[at]
                                       : __bfloat162float(static_cast<const __nv_bfloat16*>(p.teacher)[at]);
      // natural-log lse of the untempered logits
      const float nat_b = kTauIsOne ? kLn2 * lse_b : kLn2 * (mb * p.tau + log2f(sb1));
      const float nat_a = kTauIsOne ? kLn2 * lse_a : kLn2 * (ma * p.tau + log2f(sa1));
      nll_s = nat_b - dot;
      nll_t = nat_a - zt_y;
    }
  }
  if (lane == 0) {
    // cr = sum_c w(c) (O_T - O_S)[c] with w the teacher's (or, reversed, the student's) weights
    const float kl = p.reverse ? kLn2 * (-p.scale2 * (cr / sb) - lse_b + lse_a)
                               : kLn2 * (p.scale2 * (cr / sa) - lse_a + lse_b);
    p.kl[t] = on ? (kl < 0.f ? 0.f : kl) : 0.f;  // rounding may dip below 0; NaN stays NaN
    if (p.nll_s != nullptr) p.nll_s[t] = nll_s;
    if (p.nll_t != nullptr) p.nll_t[t] = nll_t;
    p.lse2_a[c] = lse_a;
    p.lse2_b[c] = lse_b;
    p.coef[c] = p.grad_scale * p.lambda / p.tau;
    if (p.coef_ce != nullptr) {
      p.coef_ce[c] = has_label ? p.grad_scale * (1.f - p.lambda) : 0.f;
      p.lse2_b1[c] = kTauIsOne ? lse_b : mb * p.tau + log2f(sb1);
    }
  }
}

struct CombineTopkParams {
  int T, d, V, topk;
  const int* plan;        // plan[2] = forward runs; the partials hold 2 slots per run
  const int* cidx;        // [T] compact row of a token (partials, lse2_b, coef*, tk_cp are indexed by it)
  const float* partials;  // [2*runs][kPFields][T]; only the student's fields are filled
  const __nv_bfloat16* hidden;
  const __nv_bfloat16* weight;
  long long ldh, ldw;
  const float* tk_val;    // [T, topk] stored teacher logits
  const int32_t* tk_idx;  // [T, topk] their vocabulary indices
  const uint8_t* loss_mask;
  const int32_t* labels;
  float scale2, tau, grad_scale, lambda;
  float* kl;
  float* nll_s;
  float* lse2_b;
  float* coef;
  float* tk_cp;           // [T, topk] coef_t * p_T(j), for the gradient tiles
  float* coef_ce;         // composite objective only (else NULL)
  float* lse2_b1;
};

// <H[t], W[c]> in fp32, one warp.
__device__ __forceinline__ float warp_dot_bf16(const __nv_bfloat16* h, const __nv_bfloat16* w, int d, int lane) {
  const uint4* h4 = reinterpret_cast<const uint4*>(h);
  const uint4* w4 = reinterpret_cast<const uint4*>(w);
  float dot = 0.f;
  for (int i = lane; i < d / 8; i += 32) {
    const uint4 a = h4[i], b = w4[i];
    dot = fmaf(bf16_lo(a.x), bf16_lo(b.x), dot);
    dot = fmaf(bf16_hi(a.x), bf16_hi(b.x), dot);
    dot = fmaf(bf16_lo(a.y), bf16_lo(b.y), dot);
    dot = fmaf(bf16_hi(a.y), bf16_hi(b.y), dot);
    dot = fmaf(bf16_lo(a.z), bf16_lo(b.z), dot);
    dot = fmaf(bf16_hi(a.z), bf16_hi(b.z), dot);
    dot = fmaf(bf16_lo(a.w), bf16_lo(b.w), dot);
    dot = fmaf(bf16_hi(a.w), bf16_hi(b.w), dot);
  }
  return warp_sum(dot);
}

// One warp per token, teacher stored as its k largest logits (Eq. 2 as printed).  Merges the
// student's partials into lse(O_S/tau), forms p_T = Softmax of the k stored logits / tau, takes
// the student logit at each stored index as the dot product <H[t], W[idx]> in fp32, and sums
//   KL = sum_j p_T(j) (log p_T(j) - (O_S[idx_j]/tau - lse)).
template <bool kTauIsOne>
__global__ void __launch_bounds__(256) kd_combine_topk_kernel(const CombineTopkParams p) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= p.T) return;
  const bool on = p.loss_mask == nullptr || p.loss_mask[t] != 0;
  if (!on) {
    if (lane == 0) {
      p.kl[t] = 0.f;
      if (p.nll_s != nullptr) p.nll_s[t] = 0.f;
    }
    return;
  }
  const int c = p.cidx[t];  // the token's compact row
  float* cp = p.tk_cp + static_cast<size_t>(c) * p.topk;
  const int nslots = 2 * p.plan[2];
  const size_t fs = static_cast<size_t>(p.T), ss = static_cast<size_t>(kPFields) * fs;
  float mb = -INFINITY;
  for (int s = lane; s < nslots; s += 32) mb = fmaxf(mb, p.partials[s * ss + kPMaxB * fs + c]);
  mb = warp_max(mb);
  float sb = 0.f, sb1 = 0.f;
  for (int s = lane; s < nslots; s += 32) {
    const float* q = p.partials + s * ss + c;
    const float db = q[kPMaxB * fs] - mb;
    sb = fmaf(q[kPSumB * fs], exp2f(db), sb);
    if (!kTauIsOne) sb1 = fmaf(q[kPSumB1 * fs], exp2f(db * p.tau), sb1);
  }
  sb = warp_sum(sb);
  if (!kTauIsOne) sb1 = warp_sum(sb1);
  const float lse_b = mb + log2f(sb);                    // base 2, of O_S * log2(e)/tau
  const float lse_b1 = kTauIsOne ? lse_b : mb * p.tau + log2f(sb1);  // same at temperature 1
  const __nv_bfloat16* h = p.hidden + static_cast<size_t>(t) * p.ldh;

  // teacher distribution on its stored support (lane j holds entry j; topk <= 32)
  const float v = lane < p.topk ? p.tk_val[static_cast<size_t>(t) * p.topk + lane] : -INFINITY;
  const float a2 = fmaxf(v, kd_cfg::kNegClamp) * p.scale2;       // base-2 scaled teacher logit
  const float ma = warp_max(lane < p.topk ? a2 : -INFINITY);
  const float ea = lane < p.topk ? exp2f(a2 - ma) : 0.f;
  const float sa = warp_sum(ea);
  const float pt = ea / sa;
  const float lse_a = ma + log2f(sa);
  float kl = 0.f;
  for (int j = 0; j < p.topk; ++j) {
    int c = p.tk_idx[static_cast<size_t>(t) * p.topk + j];
    c = c < 0 ? 0 : (c >= p.V ? p.V - 1 : c);               // indices outside [0,V) are a caller error
    const float sj = warp_dot_bf16(h, p.weight + static_cast<size_t>(c) * p.ldw, p.d, lane);
    const float ptj = __shfl_sync(0xffffffffu, pt, j), a2j = __shfl_sync(0xffffffffu, a2, j);
    // log2 p_T(j) - log2 p_S(idx_j); a zero probability contributes nothing
    if (ptj > 0.f) kl = fmaf(ptj, (a2j - lse_a) - (sj * p.scale2 - lse_b), kl);
  }
  float nll_s = 0.f;
  bool has_label = false;
  if (p.labels != nullptr) {
    const int y = p.labels[t];
    if (y >= 0 && y < p.V) {
      has_label = true;
      const float dot = warp_dot_bf16(h, p.weight + static_cast<size_t>(y) * p.ldw, p.d, lane);
      nll_s = kLn2 * lse_b1 - dot;
    }
  }
  const float coef = p.grad_scale * p.lambda / p.tau;
  if (lane < p.topk) cp[lane] = coef * pt;
  if (lane == 0) {
    kl *= kLn2;
    p.kl[t] = kl < 0.f ? 0.f : kl;
    if (p.nll_s != nullptr) p.nll_s[t] = nll_s;
    p.lse2_b[c] = lse_b;
    p.coef[c] = coef;
    if (p.coef_ce != nullptr) {
      p.coef_ce[c] = has_label ? p.grad_scale * (1.f - p.lambda) : 0.f;
      p.lse2_b1[c] = lse_b1;
    }
  }
}

// One warp per packed segment: masked sums of the per-token values and the count of
// tokens that carry a label, reduced with warp shuffles in a fixed order; also the
// token -> segment map and the validation of cu_seqlens.
__global__ void __launch_bounds__(128) segment_stats_kernel(
    int T, int S, const int32_t* __restrict__ cu, const uint8_t* __restrict__ mask,
    const int32_t* __restrict__ labels, const float* __restrict__ kl,
    const float* __restrict__ nll_s, const float* __restrict__ nll_t, float* kl_sum, float* s_sum,
    float* t_sum, int32_t* count, int32_t* seg_id, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (s >= S) return;
  const int lo = cu[s], hi = cu[s + 1];
  const bool bad = lo < 0 || hi > T || lo >= hi || (s == 0 && lo != 0) || (s == S - 1 && hi != T);
  if (bad) {
    if (lane == 0) {
      if (status != nullptr) atomicCAS(status, 0, kStatusSeq);
      if (kl_sum != nullptr) kl_sum[s] = 0.f;
      if (s_sum != nullptr) s_sum[s] = 0.f;
      if (t_sum != nullptr) t_sum[s] = 0.f;
      if (count != nullptr) count[s] = 0;
    }
    return;
  }
  float a = 0.f, b = 0.f, c = 0.f;
  int n = 0;
  for (int t = lo + lane; t < hi; t += 32) {
    const bool on = mask == nullptr || mask[t] != 0;
    const bool has = on && (labels == nullptr || labels[t] >= 0);
    if (on && kl != nullptr) a += kl[t];
    if (has) {
      if (nll_s != nullptr) b += nll_s[t];
      if (nll_t != nullptr) c += nll_t[t];
      ++n;
    }
    if (seg_id != nullptr) seg_id[t] = s;
  }
  a = warp_sum(a);
  b = warp_sum(b);
  c = warp_sum(c);
  n = warp_sum_int(n);
  if (lane == 0) {
    if (kl_sum != nullptr) kl_sum[s] = a;
    if (s_sum != nullptr) s_sum[s] = b;
    if (t_sum != nullptr) t_sum[s] = c;
    if (count != nullptr) count[s] = n;
  }
}

// One thread per sample: IFD (Eq. 3) for teacher and student from token-mean
// cross-entropies, Delta-IFD (Eq. 4), and the inclusive keep interval.
__global__ void __launch_bounds__(256) select_kernel(
    int N, int S, const int32_t* __restrict__ cond, const int32_t* __restrict__ uncond,
    const float* __restrict__ s_sum, const float* __restrict__ t_sum,
    const int32_t* __restrict__ count, float lo, float hi, int flags, float* ifd_t, float* ifd_s,
    float* delta, uint8_t* keep, int32_t* n_keep) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  int kept = 0;
  if (i < N) {
    const int c = cond[i], u = uncond[i];
    const float nan = __int_as_float(0x7fc00000);
    float it = nan, is = nan;
    if (c >= 0 && c < S && u >= 0 && u < S) {
      const int nc = count[c], nu = count[u];
      if (nc > 0 && nu > 0) {
        const float fc = static_cast<float>(nc), fu = static_cast<float>(nu);
        const float tu = __fdiv_rn(t_sum[u], fu), su = __fdiv_rn(s_sum[u], fu);
        if (tu != 0.f) it = __fdiv_rn(__fdiv_rn(t_sum[c], fc), tu);
        if (su != 0.f) is = __fdiv_rn(__fdiv_rn(s_sum[c], fc), su);
      }
    }
    const float dl = __fsub_rn(it, is);
    // what the interval tests (the filter ablation also tests the two IFDs alone) and whether
    // its ends belong to it; every comparison is false for NaN
    const float sc = (flags & 2) ? it : ((flags & 4) ? is : dl);
    bool k = ((flags & 8) ? (sc > lo) : (sc >= lo)) && ((flags & 16) ? (sc < hi) : (sc <= hi));
    if (flags & 1) k = k && (it <= 1.0f);
    if (ifd_t != nullptr) ifd_t[i] = it;
    if (ifd_s != nullptr) ifd_s[i] = is;
    if (delta != nullptr) delta[i] = dl;
    keep[i] = k ? 1 : 0;
    kept = k ? 1 : 0;
  }
  kept = warp_sum_int(kept);
  if ((threadIdx.x & 31) == 0 && kept != 0) atomicAdd(n_keep, kept);
}

// One thread per sample: perplexity of the sample's answer tokens under the student and under the
// teacher, exp(token-mean cross-entropy) (the classical filtering metric the filter ablation
// compares Delta-IFD with); NaN for a sample without such tokens or a segment index out of range.
__global__ void __launch_bounds__(256) perplexity_kernel(int N, int S, const int32_t* __restrict__ seg,
                                                        const float* __restrict__ s_sum,
                                                        const float* __restrict__ t_sum,
                                                        const int32_t* __restrict__ count,
                                                        float* ppl_s, float* ppl_t) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int c = seg[i];
  const float nan = __int_as_float(0x7fc00000);
  float ps = nan, pt = nan;
  if (c >= 0 && c < S && count[c] > 0) {
    const float n = static_cast<float>(count[c]);
    if (s_sum != nullptr) ps = expf(__fdiv_rn(s_sum[c], n));
    if (t_sum != nullptr) pt = expf(__fdiv_rn(t_sum[c], n));
  }
  if (ppl_s != nullptr) ppl_s[i] = ps;
  if (ppl_t != nullptr) ppl_t[i] = pt;
}

struct ValidateParams {
  int T, d, V, topk;
  const __nv_bfloat16* hidden;
  long long ldh;
  const void* teacher;   // dense bf16 / fp32 logits, or NULL with a top-k teacher
  int teacher_f32;
  long long ldt;
  const int32_t* tk_idx; // [T, topk] or NULL
  const uint8_t* loss_mask;
  const int32_t* labels;
  int* status;
};
constexpr int kStatusData = -10;

// Debug mode of the step: one warp per token checks what the kernels otherwise take on trust.
// Every label must be below V.  For a token that carries loss: finite hidden states; with a dense
// teacher no NaN or +inf logit and at least one finite one (a row that is entirely -inf has no
// distribution); with a top-k teacher every stored index inside [0, V).  Rows of tokens without
// loss are not read.  The first violation found sets the status word.
__global__ void __launch_bounds__(256) validate_inputs_kernel(const ValidateParams p) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= p.T) return;
  bool bad = false;
  if (p.labels != nullptr && lane == 0) bad = p.labels[t] >= p.V;
  const bool on = p.loss_mask == nullptr || p.loss_mask[t] != 0;
  if (on) {
    const __nv_bfloat16* h = p.hidden + static_cast<size_t>(t) * p.ldh;
    for (int k = lane; k < p.d; k += 32) bad |= !isfinite(__bfloat162float(h[k]));
    if (p.tk_idx != nullptr) {
      for (int j = lane; j < p.topk; j += 32) {
        const int c = p.tk_idx[static_cast<size_t>(t) * p.topk + j];
        bad |= c < 0 || c >= p.V;
      }
    } else if (p.teacher != nullptr) {
      bool support = false;
      const size_t row = static_cast<size_t>(t) * p.ldt;
      for (int c = lane; c < p.V; c += 32) {
        const float z = p.teacher_f32 ? static_cast<const float*>(p.teacher)[row + c]
                                      : __bfloat162float(static_cast<const __nv_bfloat16*>(p.teacher)[row + c]);
        bad |= isnan(z) || (isinf(z) && z > 0.f);
        support |= isfinite(z);
      }
      bad |= !__any_sync(0xffffffffu, support);
    }
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicCAS(p.status, 0, kStatusData);
}

// Self-test of the bounded-wait path, on a healthy device: one CTA of 128 threads waits, with the
// same mbar_wait the tensor kernels use, on an mbarrier that nothing ever arrives on.  When the
// (short) limit runs out the threads agree to leave through the same vote barrier the epilogue
// groups use, and the status word receives the time-out code the same way the tensor kernels
// report it.  No copy and no MMA is in flight; the kernel always terminates.
//   out[0] = status word (must be 0 on entry), out[1] = 1 if every thread's wait returned false,
//   out[2] = SM clock cycles thread 0 spent in the wait (low 31 bits)
__global__ void __launch_bounds__(128) wait_timeout_selftest_kernel(long long limit_cycles, int* out) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  const long long t0 = clock64();
  const bool okw = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_cycles));
  const long long dt = clock64() - t0;
  const bool ok = named_barrier_vote(1, 128, okw);
  const int none_ok = __syncthreads_and(okw ? 0 : 1);
  if (threadIdx.x == 0) {
    if (!ok && abort_flag != 0) atomicCAS(out, 0, kStatusTimeout);
    out[1] = none_ok;
    out[2] = static_cast<int>(dt & 0x7fffffff);
  }
}

// fp32 dH accumulator over the compact rows -> bf16 [T, ld] output by token; tokens without a
// compact row (no loss) get zeros.  8 elements per thread.
__global__ void __launch_bounds__(256) scatter_dhidden_kernel(const float* __restrict__ src,
                                                             const int* __restrict__ cidx, int T, int d,
                                                             __nv_bfloat16* dst, long long ld) {
  const long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int per_row = d / 8;
  if (i >= static_cast<long long>(T) * per_row) return;
  const int t = static_cast<int>(i / per_row), k = static_cast<int>(i % per_row) * 8;
  const int c = cidx[t];
  uint4 o = make_uint4(0u, 0u, 0u, 0u);
  if (c >= 0) {
    const float4 a = *reinterpret_cast<const float4*>(src + static_cast<size_t>(c) * d + k);
    const float4 b = *reinterpret_cast<const float4*>(src + static_cast<size_t>(c) * d + k + 4);
    o.x = pack_bf16x2(a.x, a.y);
    o.y = pack_bf16x2(a.z, a.w);
    o.z = pack_bf16x2(b.x, b.y);
    o.w = pack_bf16x2(b.z, b.w);
  }
  *reinterpret_cast<uint4*>(dst + static_cast<size_t>(t) * ld + k) = o;
}

}  // namespace npd
