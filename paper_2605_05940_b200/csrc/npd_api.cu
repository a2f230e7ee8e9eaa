// Host side of the C ABI declared in include/npd.h: argument checks, workspace
// layout, TMA descriptors and kernel launches.  Nothing here allocates device
// memory, and no problem state survives a call.  What does persist: two per-thread diagnostic
// counters, the per-device list of kernels whose shared-memory limit has been raised, and, for
// npd_kd_forward_noalloc alone, a fixed scratch array in the library image with its cached
// per-device address (which does not survive a cudaDeviceReset).
#include "../../include/npd.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <vector>

#include "gemm_sm100.cuh"
#include "kd_tile_sm100.cuh"
#include "small_kernels.cuh"

namespace {

using namespace npd;

thread_local int g_launches = 0;
thread_local long long g_h2d_bytes = 0, g_d2h_bytes = 0;  // of the last npd_kd_fwd_bwd_host call

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

PFN_cuTensorMapEncodeTiled_v12000 tensor_map_encoder() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(f);
  }();
  return fn;
}

// 2-D tensor map, 128-byte swizzle by default (swizzle64: 64-byte swizzle for boxes with 64-byte
// rows).  inner = contiguous extent (elements), outer = rows, ld = row stride (elements),
// box = {box_inner, box_outer}.
bool make_map(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t ld,
              uint32_t box_inner, uint32_t box_outer, bool f32 = false, bool swizzle = true,
              bool swizzle64 = false) {
  auto enc = tensor_map_encoder();
  if (enc == nullptr) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * (f32 ? 4 : 2)};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return enc(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
             const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             swizzle ? (swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B)
                     : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct DeviceInfo {
  int sms = 0;
  int cc_major = 0;
};
int device_info(DeviceInfo* out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return NPD_ECUDA;
  if (cudaDeviceGetAttribute(&out->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&out->cc_major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return NPD_ECUDA;
  return NPD_OK;
}

struct Plan {
  int row_blocks, vtiles, clusters;
  int nsplit_max;     // upper bound of the forward's vocabulary runs (the device picks the number)
  int chunk_cols;     // vocabulary columns per gradient chunk (multiple of 256)
  int nchunks;
  bool grads;
  size_t off_status, off_plan, off_rows, off_cidx, off_hc, off_partials, off_lse_a, off_lse_b, off_coef, off_coef_ce,
      off_lse_b1, off_tkcp, off_g, off_dh, total;
};

int make_plan(const npd_kd_args* a, int sms, Plan* pl) {
  pl->row_blocks = (a->T + 127) / 128;
  pl->vtiles = (a->V + 255) / 256;
  pl->clusters = std::max(sms / 2, 1);
  // Up to 32 runs: enough to fill the CTA pairs evenly whatever the number of row pairs turns
  // out to be; the partials cost 56 bytes per token and run.
  pl->nsplit_max = std::min(pl->vtiles, 32);
  pl->grads = a->d_hidden != nullptr || a->d_weight != nullptr;
  // Vocabulary chunks of the backward: the bf16 logit-gradient block [T, chunk_cols] is the only
  // thing that travels between the gradient tiles and the two contractions.  Default: the
  // largest chunk whose block stays within 256 MiB or a sixteenth of the teacher logits' size,
  // whichever is more (wide chunks keep the contraction units long and the number of passes
  // over the dH accumulator small), chunks of (almost) equal width.
  const long long budget = std::max<long long>(256ll << 20, static_cast<long long>(a->T) * a->V / 8);
  int max_tiles = a->grad_chunk_cols > 0
                      ? (a->grad_chunk_cols + 255) / 256
                      : static_cast<int>(std::max<long long>(8, budget / (512ll * a->T)));
  max_tiles = std::max(1, std::min(max_tiles, pl->vtiles));
  pl->nchunks = (pl->vtiles + max_tiles - 1) / max_tiles;
  const int chunk_tiles = (pl->vtiles + pl->nchunks - 1) / pl->nchunks;
  pl->chunk_cols = chunk_tiles * 256;
  pl->nchunks = (pl->vtiles + chunk_tiles - 1) / chunk_tiles;
  const int cc = pl->chunk_cols;
  size_t off = 0;
  pl->off_status = off;
  off += 1024;
  pl->off_plan = off;
  off += 1024;
  const size_t crows = static_cast<size_t>(pl->row_blocks) * 128;  // upper bound of the compact rows
  pl->off_rows = off;
  off = align_up(off + sizeof(int) * crows, 1024);
  pl->off_cidx = off;
  off = align_up(off + sizeof(int) * static_cast<size_t>(a->T), 1024);
  pl->off_hc = off;  // hidden states of the compact rows, bf16 [crows, d]
  off = align_up(off + 2 * crows * a->d, 1024);
  pl->off_partials = off;
  off = align_up(off + sizeof(float) * 2 * pl->nsplit_max * kPFields * static_cast<size_t>(a->T), 1024);
  pl->off_lse_a = off;
  off = align_up(off + sizeof(float) * a->T, 1024);
  pl->off_lse_b = off;
  off = align_up(off + sizeof(float) * a->T, 1024);
  pl->off_coef = off;
  off = align_up(off + sizeof(float) * a->T, 1024);
  pl->off_coef_ce = pl->off_lse_b1 = off;
  if (a->flags & NPD_KD_COMPOSITE_LOSS) {
    pl->off_coef_ce = off;
    off = align_up(off + sizeof(float) * a->T, 1024);
    pl->off_lse_b1 = off;
    off = align_up(off + sizeof(float) * a->T, 1024);
  }
  pl->off_tkcp = off;
  if (a->topk > 0) off = align_up(off + sizeof(float) * static_cast<size_t>(a->T) * a->topk, 1024);
  pl->off_g = off;
  pl->off_dh = off;
  if (pl->grads) {
    off = align_up(off + 2 * crows * cc, 1024);
    pl->off_dh = off;  // fp32 dH accumulator over the compact rows
    off = align_up(off + sizeof(float) * crows * a->d, 1024);
  }
  pl->total = off;
  return NPD_OK;
}

int check_args(const npd_kd_args* a, bool need_pointers) {
  if (a == nullptr || a->size != sizeof(npd_kd_args)) return NPD_EINVAL;
  if (a->T < 1 || a->d < 1 || a->V < 1) return NPD_EINVAL;
  if (!(a->temperature > 0.f) || !std::isfinite(a->temperature)) return NPD_EINVAL;
  if (a->teacher_dtype != NPD_DTYPE_BF16 && a->teacher_dtype != NPD_DTYPE_F32) return NPD_EINVAL;
  const bool tf32 = a->teacher_dtype == NPD_DTYPE_F32;
  if (a->d_weight_dtype != NPD_DTYPE_BF16 && a->d_weight_dtype != NPD_DTYPE_F32) return NPD_EINVAL;
  if (a->grad_chunk_cols < 0 || a->n_phase_events < 0) return NPD_EINVAL;
  if (a->d % 64 != 0) return NPD_ESHAPE;
  const bool sparse = a->topk != 0;
  if (sparse && (a->topk < 0 || a->nll_teacher != nullptr)) return NPD_EINVAL;
  if (sparse && a->topk > kd_cfg::kMaxTopK) return NPD_EUNSUPPORTED;
  if (a->ldh < a->d || a->ldw < a->d || (!sparse && a->ldt < a->V)) return NPD_ESHAPE;
  if (a->cu_seqlens != nullptr && (a->S < 1 || a->S > a->T)) return NPD_ESHAPE;
  if ((a->ldh % 8) || (a->ldw % 8) || (!sparse && (a->ldt % (tf32 ? 4 : 8)))) return NPD_EALIGN;
  if ((a->d_hidden == nullptr) != (a->d_weight == nullptr)) return NPD_EINVAL;
  if ((a->flags & NPD_KD_ACCUMULATE_DW) && a->d_weight_dtype != NPD_DTYPE_F32) return NPD_EINVAL;
  if ((a->flags & NPD_KD_REVERSE_KL) && (a->d_hidden != nullptr || a->topk != 0)) return NPD_EINVAL;
  if (a->flags & NPD_KD_COMPOSITE_LOSS) {
    if (!(a->kd_lambda >= 0.f && a->kd_lambda <= 1.f)) return NPD_EINVAL;
    if (need_pointers && a->labels == nullptr) return NPD_EINVAL;
  }
  if (!need_pointers) return NPD_OK;
  if (a->hidden == nullptr || a->weight == nullptr || a->kl == nullptr) return NPD_EINVAL;
  if (sparse ? (a->topk_values == nullptr || a->topk_indices == nullptr) : (a->teacher == nullptr))
    return NPD_EINVAL;
  if (!aligned16(a->hidden) || !aligned16(a->weight) || (!sparse && !aligned16(a->teacher)) ||
      !aligned16(a->d_hidden) || !aligned16(a->d_weight))
    return NPD_EALIGN;
  if (a->d_weight != nullptr && a->d_weight_dtype == NPD_DTYPE_F32 && (a->ldw % 4)) return NPD_EALIGN;
  return NPD_OK;
}

// Records the caller's optional phase events in order.
struct PhaseRecorder {
  void* const* ev;
  int n, next;
  cudaStream_t st;
  void mark() {
    if (ev != nullptr && next < n && ev[next] != nullptr) cudaEventRecord(static_cast<cudaEvent_t>(ev[next]), st);
    ++next;
  }
};

// Raises a kernel's dynamic shared-memory limit; done once per kernel and device.
template <typename K>
int set_smem(K kernel, int bytes) {
  static std::mutex mu;
  static std::vector<std::pair<const void*, int>> done;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return NPD_ECUDA;
  const void* key = reinterpret_cast<const void*>(kernel);
  std::lock_guard<std::mutex> lock(mu);
  for (const auto& e : done)
    if (e.first == key && e.second == dev) return NPD_OK;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
    return NPD_ECUDA;
  done.emplace_back(key, dev);
  return NPD_OK;
}

// Launch with (pdl) or without the programmatic-dependent-launch attribute: with it, the blocks
// of this kernel may be scheduled and run their prologue while the kernel before it in the stream
// is still draining; they wait for that kernel's completion inside (griddepcontrol.wait).
template <typename... P, typename... A>
cudaError_t launch_ex(void (*kernel)(P...), int grid, int threads, int smem, cudaStream_t st, bool pdl,
                      A&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(static_cast<unsigned>(threads));
  cfg.dynamicSmemBytes = static_cast<size_t>(smem);
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<P>(args)...);
}

struct GemmOperands {
  const void* A;
  long long lda;
  const void* B;
  long long ldb;
  void* out;
  long long ldo;
};

// The two backward contractions of one vocabulary chunk of `cols` columns.  Everything lives on
// the compact rows (their number is only known on the device): the logit-gradient block, the
// gathered hidden states and the fp32 dH accumulator.
void chunk_problems(int d, int cols, bool dw_f32, bool dw_accumulate, GemmProblem* pr) {
  // dW[col0 .. col0+cols) = G_chunk^T Hc      (M = vocabulary rows, N = d, K = compact rows)
  pr[0] = GemmProblem{};
  pr[0].M = cols;
  pr[0].N = d;
  pr[0].dyn_k = 1;
  pr[0].a_mn = 1;
  pr[0].b_mn = 1;
  pr[0].k_splits = 1;
  pr[0].out_f32 = dw_f32;
  pr[0].out_reduce = dw_accumulate ? 1 : 0;
  // dH += G_chunk W[col0 .. col0+cols)        (M = compact rows, N = d, K = the chunk's columns)
  pr[1] = GemmProblem{};
  pr[1].dyn_m = 1;
  pr[1].N = d;
  pr[1].K = cols;
  pr[1].b_mn = 1;
  pr[1].k_splits = 1;
  pr[1].stream_k = 1;
  pr[1].out_f32 = 1;
  pr[1].out_reduce = 1;
}

// One launch for one or two problems (see gemm_sm100.cuh for how the units are dealt).
// An extent only known on the device (dyn_m / dyn_k) is 128 * max_blocks as far as the maps go.
int launch_gemm(int nprob, const GemmProblem* pr, const GemmOperands* ops, const int* nblocks,
                int max_blocks, int* status, int sms, cudaStream_t st, bool pdl = false) {
  using namespace gemm_cfg;
  CUtensorMap maps[6];
  GemmParams gp{};
  long long units = 0;
  for (int i = 0; i < 2; ++i) {
    const int j = i < nprob ? i : 0;  // an unused slot repeats problem 0's (valid) maps
    const GemmProblem& g = pr[j];
    // extents as the maps see them: device-side dimensions take their upper bound
    const uint64_t am = g.dyn_m ? 128ull * max_blocks : g.M, ak = g.dyn_k ? 128ull * max_blocks : g.K;
    const uint64_t bk = ak, om = am;
    const bool oka = g.a_mn ? make_map(&maps[3 * i], ops[j].A, am, ak, ops[j].lda, 64, 64)
                            : make_map(&maps[3 * i], ops[j].A, ak, am, ops[j].lda, 64, BM);
    const bool okb = g.b_mn ? make_map(&maps[3 * i + 1], ops[j].B, g.N, bk, ops[j].ldb, 64, 64)
                            : make_map(&maps[3 * i + 1], ops[j].B, bk, g.N, ops[j].ldb, 64, BNS / 2);
    // output sub-tiles: 128 rows x 64 bytes, 64-byte swizzle
    const bool oko = make_map(&maps[3 * i + 2], ops[j].out, g.N, om, ops[j].ldo, g.out_f32 ? 16 : 32, BM,
                              g.out_f32 != 0, true, true);
    if (!oka || !okb || !oko) return NPD_ECUDA;
    gp.pr[i] = g;
    if (i < nprob)
      units += static_cast<long long>((am + PM - 1) / PM) * ((g.N + BN - 1) / BN) * g.k_splits;
  }
  gp.nprob = nprob;
  gp.nblocks = nblocks;
  gp.status = status;
  const int pairs = static_cast<int>(std::max<long long>(1, std::min<long long>(units, std::max(sms / 2, 1))));
  if (set_smem(gemm_bf16_kernel, SMEM_BYTES) != NPD_OK) return NPD_ECUDA;
  const cudaError_t e = launch_ex(gemm_bf16_kernel, 2 * pairs, THREADS, SMEM_BYTES, st, pdl, maps[0], maps[1],
                                  maps[2], maps[3], maps[4], maps[5], gp);
  ++g_launches;
  return e == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

template <int kMode>
int launch_kd_tile(bool tau_one, bool composite, bool sparse, bool tf32, const CUtensorMap& mh, const CUtensorMap& mw, const CUtensorMap& mt,
                   const CUtensorMap& mg, const KdTileParams& kp, int sms, cudaStream_t st, bool pdl) {
  using namespace kd_cfg;
  composite = composite && kMode == kGradient;  // the forward does not depend on the objective's mix
  auto k = kd_tile_kernel<kMode, true, false, false, false>;
  if (sparse) {
    if (!composite) k = tau_one ? kd_tile_kernel<kMode, true, false, true, false> : kd_tile_kernel<kMode, false, false, true, false>;
    else k = tau_one ? kd_tile_kernel<kMode, true, true, true, false> : kd_tile_kernel<kMode, false, true, true, false>;
  } else if (tf32) {
    if (!composite) k = tau_one ? kd_tile_kernel<kMode, true, false, false, true> : kd_tile_kernel<kMode, false, false, false, true>;
    else k = tau_one ? kd_tile_kernel<kMode, true, true, false, true> : kd_tile_kernel<kMode, false, true, false, true>;
  } else {
    if (!composite) k = tau_one ? kd_tile_kernel<kMode, true, false, false, false> : kd_tile_kernel<kMode, false, false, false, false>;
    else k = tau_one ? kd_tile_kernel<kMode, true, true, false, false> : kd_tile_kernel<kMode, false, true, false, false>;
  }
  if (set_smem(k, Layout<kMode>::SMEM_BYTES) != NPD_OK) return NPD_ECUDA;
  // the number of units is only known on the device: always one CTA pair per two SMs
  const int grid = 2 * std::max(sms / 2, 1);
  const cudaError_t e = launch_ex(k, grid, THREADS, Layout<kMode>::SMEM_BYTES, st, pdl, mh, mw, mt, mg, kp);
  ++g_launches;
  return e == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

}  // namespace

extern "C" {

const char* npd_strerror(int status) {
  switch (status) {
    case NPD_OK: return "ok";
    case NPD_EINVAL: return "invalid argument";
    case NPD_ESHAPE: return "unsupported shape or stride";
    case NPD_EALIGN: return "pointer or stride not 16-byte aligned";
    case NPD_ESEQ: return "malformed cu_seqlens";
    case NPD_EARCH: return "device is not compute capability 10.x";
    case NPD_EWORKSPACE: return "workspace missing, misaligned or too small";
    case NPD_ECUDA: return "CUDA call failed";
    case NPD_ETIMEOUT: return "bounded device-side wait expired";
    case NPD_EUNSUPPORTED: return "option not implemented";
    case NPD_EDATA: return "input data the step may not be given (debug checks)";
    default: return "unknown status";
  }
}

int npd_last_launch_count(void) { return g_launches; }

int npd_last_copy_bytes(int64_t* h2d_bytes, int64_t* d2h_bytes) {
  if (h2d_bytes == nullptr || d2h_bytes == nullptr) return NPD_EINVAL;
  *h2d_bytes = g_h2d_bytes;
  *d2h_bytes = g_d2h_bytes;
  return NPD_OK;
}

int npd_workspace_bytes(const npd_kd_args* args, size_t* out_bytes) {
  if (out_bytes == nullptr) return NPD_EINVAL;
  int rc = check_args(args, false);
  if (rc != NPD_OK) return rc;
  DeviceInfo di;
  if ((rc = device_info(&di)) != NPD_OK) return rc;
  Plan pl;
  make_plan(args, di.sms, &pl);
  *out_bytes = pl.total;
  return NPD_OK;
}

int npd_kd_fwd_bwd(const npd_kd_args* a, void* cuda_stream) {
  g_launches = 0;
  int rc = check_args(a, true);
  if (rc != NPD_OK) return rc;
  DeviceInfo di;
  if ((rc = device_info(&di)) != NPD_OK) return rc;
  if (di.cc_major != 10) return NPD_EARCH;
  Plan pl;
  make_plan(a, di.sms, &pl);
  if (a->workspace == nullptr || (reinterpret_cast<uintptr_t>(a->workspace) & 1023u) ||
      a->workspace_bytes < pl.total)
    return NPD_EWORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = static_cast<uint8_t*>(a->workspace);
  int* status = reinterpret_cast<int*>(ws + pl.off_status);
  int* plan = reinterpret_cast<int*>(ws + pl.off_plan);
  int* rows = reinterpret_cast<int*>(ws + pl.off_rows);
  int* cidx = reinterpret_cast<int*>(ws + pl.off_cidx);
  __nv_bfloat16* hc = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_hc);
  const uint64_t crows = static_cast<uint64_t>(pl.row_blocks) * 128;
  float* partials = reinterpret_cast<float*>(ws + pl.off_partials);
  float* lse_a = reinterpret_cast<float*>(ws + pl.off_lse_a);
  float* lse_b = reinterpret_cast<float*>(ws + pl.off_lse_b);
  float* coef = reinterpret_cast<float*>(ws + pl.off_coef);
  const bool composite = (a->flags & NPD_KD_COMPOSITE_LOSS) != 0;
  float* coef_ce = composite ? reinterpret_cast<float*>(ws + pl.off_coef_ce) : nullptr;
  float* lse_b1 = composite ? reinterpret_cast<float*>(ws + pl.off_lse_b1) : nullptr;
  if (cudaMemsetAsync(status, 0, 64, st) != cudaSuccess) return NPD_ECUDA;
  PhaseRecorder rec{a->phase_events, a->n_phase_events, 0, st};

  const bool pdl = (a->flags & NPD_KD_SERIALIZE_LAUNCHES) == 0;
  const bool tau_one = a->temperature == 1.0f;
  const float scale2 = 1.4426950408889634f / a->temperature;

  const bool sparse = a->topk > 0;  // teacher stored as its top-k logits per token
  const bool tf32 = !sparse && a->teacher_dtype == NPD_DTYPE_F32;
  float* tk_cp = reinterpret_cast<float*>(ws + pl.off_tkcp);
  CUtensorMap mh, mw, mt;
  // H is read as its compact copy; the teacher by four-row gathers (box one row high)
  if (!make_map(&mh, hc, a->d, crows, a->d, 64, 128) ||
      !make_map(&mw, a->weight, a->d, a->V, a->ldw, 64, 128))
    return NPD_ECUDA;
  if (sparse) {
    mt = mh;  // never used: no teacher tiles are streamed
  } else if (!make_map(&mt, a->teacher, a->V, a->T, a->ldt, tf32 ? 32 : 64, 1, tf32)) {
    return NPD_ECUDA;
  }

  // cu_seqlens is validated on the device; the result lands in the status word.
  if (a->cu_seqlens != nullptr) {
    segment_stats_kernel<<<(a->S + 3) / 4, 128, 0, st>>>(a->T, a->S, a->cu_seqlens, nullptr, nullptr,
                                                        nullptr, nullptr, nullptr, nullptr, nullptr,
                                                        nullptr, nullptr, nullptr, status);
    ++g_launches;
  }

  if (a->flags & NPD_KD_DEBUG_CHECKS) {
    ValidateParams vp{};
    vp.T = a->T;
    vp.d = a->d;
    vp.V = a->V;
    vp.topk = a->topk;
    vp.hidden = static_cast<const __nv_bfloat16*>(a->hidden);
    vp.ldh = a->ldh;
    vp.teacher = sparse ? nullptr : a->teacher;
    vp.teacher_f32 = tf32 ? 1 : 0;
    vp.ldt = a->ldt;
    vp.tk_idx = sparse ? a->topk_indices : nullptr;
    vp.loss_mask = a->loss_mask;
    vp.labels = a->labels;
    vp.status = status;
    validate_inputs_kernel<<<(a->T + 7) / 8, 256, 0, st>>>(vp);
    ++g_launches;
  }

  // ---- number the tokens with loss (compact rows) and gather their hidden states; everything
  // below works on the compact rows only ----
  plan_rows_kernel<<<1, 1024, 0, st>>>(a->T, a->loss_mask, pl.vtiles, pl.nsplit_max, pl.clusters, plan, rows,
                                       cidx);
  gather_hidden_rows_kernel<<<2 * di.sms, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(a->hidden), a->ldh,
                                                        a->d, plan, rows, hc);
  g_launches += 2;
  if (cudaGetLastError() != cudaSuccess) return NPD_ECUDA;

  rec.mark();
  // ---- forward: statistics per (pair of row blocks, vocabulary run), then the per-token merge ----
  KdTileParams kp{};
  kp.T = a->T;
  kp.V = a->V;
  kp.ksteps = a->d / 64;
  kp.plan = plan;
  kp.rows = rows;
  // a group's H rows (256 x d bf16 per pair) should fill at most a quarter of a 128 MB L2
  kp.group_pairs = static_cast<int>(std::max<long long>(4, (32ll << 20) / (512ll * a->d)));
  kp.vt_begin = 0;
  kp.vt_count = pl.vtiles;
  kp.scale2 = scale2;
  kp.tau = a->temperature;
  kp.partials = partials;
  kp.reverse = (a->flags & NPD_KD_REVERSE_KL) ? 1 : 0;
  kp.status = status;
  if ((rc = launch_kd_tile<kForward>(tau_one, false, sparse, tf32, mh, mw, mt, mt, kp, di.sms, st, pdl)) != NPD_OK) return rc;
  rec.mark();

  if (sparse) {
    CombineTopkParams tp{};
    tp.T = a->T;
    tp.d = a->d;
    tp.V = a->V;
    tp.topk = a->topk;
    tp.plan = plan;
    tp.cidx = cidx;
    tp.partials = partials;
    tp.hidden = static_cast<const __nv_bfloat16*>(a->hidden);
    tp.weight = static_cast<const __nv_bfloat16*>(a->weight);
    tp.ldh = a->ldh;
    tp.ldw = a->ldw;
    tp.tk_val = a->topk_values;
    tp.tk_idx = a->topk_indices;
    tp.loss_mask = a->loss_mask;
    tp.labels = a->labels;
    tp.scale2 = scale2;
    tp.tau = a->temperature;
    tp.grad_scale = a->grad_scale;
    tp.lambda = composite ? a->kd_lambda : 1.f;
    tp.kl = a->kl;
    tp.nll_s = a->nll_student;
    tp.lse2_b = lse_b;
    tp.coef = coef;
    tp.tk_cp = tk_cp;
    tp.coef_ce = coef_ce;
    tp.lse2_b1 = lse_b1;
    if (tau_one)
      kd_combine_topk_kernel<true><<<(a->T + 7) / 8, 256, 0, st>>>(tp);
    else
      kd_combine_topk_kernel<false><<<(a->T + 7) / 8, 256, 0, st>>>(tp);
  }
  CombineParams cp{};
  cp.T = a->T;
  cp.d = a->d;
  cp.V = a->V;
  cp.plan = plan;
  cp.cidx = cidx;
  cp.partials = partials;
  cp.hidden = static_cast<const __nv_bfloat16*>(a->hidden);
  cp.weight = static_cast<const __nv_bfloat16*>(a->weight);
  cp.teacher = a->teacher;
  cp.teacher_f32 = tf32 ? 1 : 0;
  cp.ldh = a->ldh;
  cp.ldw = a->ldw;
  cp.ldt = a->ldt;
  cp.loss_mask = a->loss_mask;
  cp.labels = a->labels;
  cp.scale2 = scale2;
  cp.tau = a->temperature;
  cp.grad_scale = a->grad_scale;
  cp.kl = a->kl;
  cp.nll_s = a->nll_student;
  cp.nll_t = a->nll_teacher;
  cp.lse2_a = lse_a;
  cp.lse2_b = lse_b;
  cp.coef = coef;
  cp.lambda = composite ? a->kd_lambda : 1.f;
  cp.reverse = kp.reverse;
  cp.coef_ce = coef_ce;
  cp.lse2_b1 = lse_b1;
  if (sparse) {
    // merged above
  } else if (tau_one) {
    kd_combine_kernel<true><<<(a->T + 7) / 8, 256, 0, st>>>(cp);
  } else {
    kd_combine_kernel<false><<<(a->T + 7) / 8, 256, 0, st>>>(cp);
  }
  ++g_launches;
  if (cudaGetLastError() != cudaSuccess) return NPD_ECUDA;
  rec.mark();
  if (!pl.grads) return NPD_OK;

  // ---- backward: per vocabulary chunk, gradient tiles -> scratch -> dW rows and dH partial ----
  __nv_bfloat16* gbuf = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_g);
  float* dh_acc = reinterpret_cast<float*>(ws + pl.off_dh);
  const long long ldg = pl.chunk_cols;
  if (cudaMemsetAsync(dh_acc, 0, sizeof(float) * crows * a->d, st) != cudaSuccess) return NPD_ECUDA;
  for (int c = 0; c < pl.nchunks; ++c) {
    const int col0 = c * pl.chunk_cols;
    const int cols = std::min(pl.chunk_cols, a->V - col0);  // columns of this chunk inside V
    if (cols <= 0) break;
    const int cols_pad = std::min(pl.chunk_cols, pl.vtiles * 256 - col0);
    CUtensorMap mg;
    // gradient sub-tiles: 64 columns in the teacher's swizzled layout, or (fp32 teacher) 32 plain
    if (!(tf32 ? make_map(&mg, gbuf, cols_pad, crows, ldg, 32, 128, false, false)
               : make_map(&mg, gbuf, cols_pad, crows, ldg, 64, 128)))
      return NPD_ECUDA;
    KdTileParams gp = kp;
    gp.vt_begin = col0 / 256;
    gp.vt_count = cols_pad / 256;
    gp.partials = nullptr;
    gp.lse2_a = lse_a;
    gp.lse2_b = lse_b;
    gp.coef = coef;
    gp.coef_ce = coef_ce;
    gp.lse2_b1 = lse_b1;
    gp.labels = a->labels;
    gp.tk_idx = a->topk_indices;
    gp.tk_cp = tk_cp;
    gp.topk = a->topk;
    gp.g_col0 = col0;
    if ((rc = launch_kd_tile<kGradient>(tau_one, composite, sparse, tf32, mh, mw, mt, mg, gp, di.sms, st, pdl)) != NPD_OK) return rc;
    rec.mark();

    GemmProblem pr[2] = {};
    GemmOperands ops[2] = {};
    chunk_problems(a->d, cols, a->d_weight_dtype == NPD_DTYPE_F32, (a->flags & NPD_KD_ACCUMULATE_DW) != 0, pr);
    void* dw_rows = pr[0].out_f32
                        ? static_cast<void*>(static_cast<float*>(a->d_weight) + static_cast<size_t>(col0) * a->ldw)
                        : static_cast<void*>(static_cast<__nv_bfloat16*>(a->d_weight) +
                                             static_cast<size_t>(col0) * a->ldw);
    ops[0] = {gbuf, ldg, hc, a->d, dw_rows, a->ldw};
    const __nv_bfloat16* w_rows = static_cast<const __nv_bfloat16*>(a->weight) + static_cast<size_t>(col0) * a->ldw;
    ops[1] = {gbuf, ldg, w_rows, a->ldw, dh_acc, a->d};
    if ((rc = launch_gemm(2, pr, ops, plan, pl.row_blocks, status, di.sms, st, pdl)) != NPD_OK) return rc;
    rec.mark();
  }
  {
    // compact fp32 rows -> bf16 rows of the tokens; tokens without loss get zeros
    const long long n = static_cast<long long>(a->T) * (a->d / 8);
    scatter_dhidden_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, st>>>(
        dh_acc, cidx, a->T, a->d, static_cast<__nv_bfloat16*>(a->d_hidden), a->ldh);
    ++g_launches;
    if (cudaGetLastError() != cudaSuccess) return NPD_ECUDA;
    rec.mark();
  }
  return NPD_OK;
}

int npd_phase_count(const npd_kd_args* args, int32_t* out_groups, int32_t* out_chunks) {
  if (out_groups == nullptr) return NPD_EINVAL;
  int rc = check_args(args, false);
  if (rc != NPD_OK) return rc;
  DeviceInfo di;
  if ((rc = device_info(&di)) != NPD_OK) return rc;
  Plan pl;
  make_plan(args, di.sms, &pl);
  int chunks = 0;
  if (pl.grads)
    for (int c = 0; c < pl.nchunks; ++c)
      if (args->V - c * pl.chunk_cols > 0) ++chunks;
  *out_groups = 2 + 2 * chunks + (pl.grads ? 1 : 0);
  if (out_chunks != nullptr) *out_chunks = chunks;
  return NPD_OK;
}

int npd_kd_fwd_bwd_host(const npd_kd_args* host, const npd_kd_args* dev, void* cuda_stream) {
  return npd_kd_fwd_bwd_host_streams(host, dev, cuda_stream, cuda_stream);
}

int npd_kd_fwd_bwd_host_streams(const npd_kd_args* host, const npd_kd_args* dev, void* copy_stream,
                                void* cuda_stream) {
  if (host == nullptr || dev == nullptr || host->size != sizeof(npd_kd_args)) return NPD_EINVAL;
  int rc = check_args(dev, true);
  if (rc != NPD_OK) return rc;
  if (host->T != dev->T || host->d != dev->d || host->V != dev->V) return NPD_EINVAL;
  if (host->hidden == nullptr || host->kl == nullptr || host->topk != dev->topk) return NPD_EINVAL;
  if (dev->topk > 0 ? (host->topk_values == nullptr || host->topk_indices == nullptr)
                    : (host->teacher == nullptr))
    return NPD_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);  // kernels and the copies back
  cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);  // the copies in
  const size_t T = dev->T;
  bool ok = true;
  g_h2d_bytes = g_d2h_bytes = 0;
  // With a copy stream of its own: the copies in start once everything queued so far on the
  // compute stream (the last user of these staging buffers) is done, and the kernels start once
  // the copies are.  Copies of different calls queue up behind each other on the copy stream
  // instead of sharing the link, so a call's kernels overlap the next call's copies.
  const bool two_streams = cs != st;
  cudaEvent_t ev = nullptr;
  if (two_streams) {
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return NPD_ECUDA;
    ok &= cudaEventRecord(ev, st) == cudaSuccess;
    ok &= cudaStreamWaitEvent(cs, ev, 0) == cudaSuccess;
  }
  // Rows of tokens without loss are never read by the kernels, so only the stretches of rows
  // that carry loss are copied (a batch with masked prompts moves that much less over PCIe).
  // With a mask that would take too many separate copies, everything is copied.
  std::vector<std::pair<size_t, size_t>> runs;  // [first row, end row)
  const bool have_mask = host->loss_mask != nullptr && dev->loss_mask != nullptr;
  if (have_mask) {
    size_t t = 0;
    while (t < T && runs.size() <= 1024) {
      while (t < T && host->loss_mask[t] == 0) ++t;
      const size_t a = t;
      while (t < T && host->loss_mask[t] != 0) ++t;
      if (t > a) runs.emplace_back(a, t);
    }
  }
  if (!have_mask || runs.size() > 1024) runs.assign(1, std::make_pair(size_t{0}, T));
  auto copy_rows = [&](const void* dst, long long ldd, const void* src, long long lds, size_t row_bytes,
                       size_t esize) {
    for (const auto& r : runs) {
      const size_t n = r.second - r.first;
      ok &= cudaMemcpy2DAsync(static_cast<char*>(const_cast<void*>(dst)) + r.first * ldd * esize, ldd * esize,
                              static_cast<const char*>(src) + r.first * lds * esize, lds * esize, row_bytes,
                              n, cudaMemcpyHostToDevice, cs) == cudaSuccess;
      g_h2d_bytes += static_cast<long long>(row_bytes * n);
    }
  };
  copy_rows(dev->hidden, dev->ldh, host->hidden, host->ldh, static_cast<size_t>(dev->d) * 2, 2);
  if (dev->topk > 0) {
    copy_rows(dev->topk_values, dev->topk, host->topk_values, dev->topk, sizeof(float) * dev->topk, sizeof(float));
    copy_rows(dev->topk_indices, dev->topk, host->topk_indices, dev->topk, sizeof(int32_t) * dev->topk,
              sizeof(int32_t));
  } else {
    const size_t te = dev->teacher_dtype == NPD_DTYPE_F32 ? 4 : 2;
    copy_rows(dev->teacher, dev->ldt, host->teacher, host->ldt, static_cast<size_t>(dev->V) * te, te);
  }
  if (dev->cu_seqlens != nullptr && host->cu_seqlens != nullptr) {
    ok &= cudaMemcpyAsync(const_cast<int32_t*>(dev->cu_seqlens), host->cu_seqlens,
                          sizeof(int32_t) * (dev->S + 1), cudaMemcpyHostToDevice, cs) == cudaSuccess;
    g_h2d_bytes += static_cast<long long>(sizeof(int32_t)) * (dev->S + 1);
  }
  if (have_mask) {
    ok &= cudaMemcpyAsync(const_cast<uint8_t*>(dev->loss_mask), host->loss_mask, T,
                          cudaMemcpyHostToDevice, cs) == cudaSuccess;
    g_h2d_bytes += static_cast<long long>(T);
  }
  if (dev->labels != nullptr && host->labels != nullptr) {
    ok &= cudaMemcpyAsync(const_cast<int32_t*>(dev->labels), host->labels, sizeof(int32_t) * T,
                          cudaMemcpyHostToDevice, cs) == cudaSuccess;
    g_h2d_bytes += static_cast<long long>(sizeof(int32_t) * T);
  }
  if (two_streams) {
    ok &= cudaEventRecord(ev, cs) == cudaSuccess;
    ok &= cudaStreamWaitEvent(st, ev, 0) == cudaSuccess;
    cudaEventDestroy(ev);  // released once the recorded work has passed it
  }
  if (!ok) return NPD_ECUDA;
  if ((rc = npd_kd_fwd_bwd(dev, cuda_stream)) != NPD_OK) return rc;
  ok &= cudaMemcpyAsync(host->kl, dev->kl, sizeof(float) * T, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  g_d2h_bytes += static_cast<long long>(sizeof(float) * T);
  if (host->nll_student != nullptr && dev->nll_student != nullptr) {
    ok &= cudaMemcpyAsync(host->nll_student, dev->nll_student, sizeof(float) * T,
                          cudaMemcpyDeviceToHost, st) == cudaSuccess;
    g_d2h_bytes += static_cast<long long>(sizeof(float) * T);
  }
  if (host->nll_teacher != nullptr && dev->nll_teacher != nullptr) {
    ok &= cudaMemcpyAsync(host->nll_teacher, dev->nll_teacher, sizeof(float) * T,
                          cudaMemcpyDeviceToHost, st) == cudaSuccess;
    g_d2h_bytes += static_cast<long long>(sizeof(float) * T);
  }
  return ok ? NPD_OK : NPD_ECUDA;
}

int npd_segment_stats(int32_t T, int32_t S, const int32_t* cu_seqlens, const uint8_t* loss_mask,
                      const int32_t* labels, const float* kl, const float* nll_student,
                      const float* nll_teacher, float* kl_sum, float* nll_s_sum, float* nll_t_sum,
                      int32_t* count, int32_t* seg_id, int32_t* status, void* cuda_stream) {
  if (T < 1 || S < 1 || cu_seqlens == nullptr) return NPD_EINVAL;
  if (S > T) return NPD_ESHAPE;
  if ((kl == nullptr) != (kl_sum == nullptr) || (nll_student == nullptr) != (nll_s_sum == nullptr) ||
      (nll_teacher == nullptr) != (nll_t_sum == nullptr))
    return NPD_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  segment_stats_kernel<<<(S + 3) / 4, 128, 0, st>>>(T, S, cu_seqlens, loss_mask, labels, kl,
                                                    nll_student, nll_teacher, kl_sum, nll_s_sum,
                                                    nll_t_sum, count, seg_id, status);
  return cudaGetLastError() == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

int npd_select(int32_t N, const int32_t* cond_seg, const int32_t* uncond_seg, const float* nll_s_sum,
               const float* nll_t_sum, const int32_t* count, int32_t S, float lo, float hi,
               int32_t flags, float* ifd_teacher, float* ifd_student, float* delta, uint8_t* keep,
               int32_t* n_keep, void* cuda_stream) {
  if (N < 1 || S < 1 || cond_seg == nullptr || uncond_seg == nullptr || nll_s_sum == nullptr ||
      nll_t_sum == nullptr || count == nullptr || keep == nullptr || n_keep == nullptr)
    return NPD_EINVAL;
  if (std::isnan(lo) || std::isnan(hi)) return NPD_EINVAL;
  if ((flags & NPD_SELECT_SCORE_IFD_TEACHER) && (flags & NPD_SELECT_SCORE_IFD_STUDENT)) return NPD_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(n_keep, 0, sizeof(int32_t), st) != cudaSuccess) return NPD_ECUDA;
  select_kernel<<<(N + 255) / 256, 256, 0, st>>>(N, S, cond_seg, uncond_seg, nll_s_sum, nll_t_sum, count,
                                                 lo, hi, flags, ifd_teacher, ifd_student, delta, keep,
                                                 n_keep);
  return cudaGetLastError() == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

int npd_pack_sequences(int32_t N, const int32_t* lengths, const uint8_t* keep, int32_t capacity,
                       int32_t* order, int32_t* row_of, int32_t* cu_seqlens, int32_t* row_ptr,
                       int32_t* n_placed, int32_t* n_rows) {
  if (N < 0 || capacity < 1 || (N > 0 && lengths == nullptr) || order == nullptr || row_of == nullptr ||
      cu_seqlens == nullptr || row_ptr == nullptr || n_placed == nullptr || n_rows == nullptr)
    return NPD_EINVAL;
  std::vector<int32_t> cand;
  cand.reserve(N);
  for (int32_t i = 0; i < N; ++i)
    if ((keep == nullptr || keep[i] != 0) && lengths[i] > 0) cand.push_back(i);
  auto len = [&](int32_t i) { return std::min(lengths[i], capacity); };
  std::stable_sort(cand.begin(), cand.end(), [&](int32_t a, int32_t b) { return len(a) > len(b); });
  std::vector<int32_t> room;                       // free tokens of every open row
  std::vector<std::vector<int32_t>> members;       // samples of every row, in placing order
  for (int32_t i : cand) {
    const int32_t n = len(i);
    size_t r = 0;
    while (r < room.size() && room[r] < n) ++r;    // first row with room
    if (r == room.size()) {
      room.push_back(capacity);
      members.emplace_back();
    }
    room[r] -= n;
    members[r].push_back(i);
  }
  int32_t j = 0;
  cu_seqlens[0] = 0;
  for (size_t r = 0; r < members.size(); ++r) {
    row_ptr[r] = j;
    for (int32_t i : members[r]) {
      order[j] = i;
      row_of[j] = static_cast<int32_t>(r);
      cu_seqlens[j + 1] = cu_seqlens[j] + len(i);
      ++j;
    }
  }
  row_ptr[members.size()] = j;
  *n_placed = j;
  *n_rows = static_cast<int32_t>(members.size());
  return NPD_OK;
}

int npd_perplexity(int32_t N, const int32_t* seg, const float* nll_s_sum, const float* nll_t_sum,
                   const int32_t* count, int32_t S, float* ppl_student, float* ppl_teacher,
                   void* cuda_stream) {
  if (N < 1 || S < 1 || seg == nullptr || count == nullptr) return NPD_EINVAL;
  if ((ppl_student != nullptr && nll_s_sum == nullptr) || (ppl_teacher != nullptr && nll_t_sum == nullptr) ||
      (ppl_student == nullptr && ppl_teacher == nullptr))
    return NPD_EINVAL;
  perplexity_kernel<<<(N + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      N, S, seg, nll_s_sum, nll_t_sum, count, ppl_student, ppl_teacher);
  return cudaGetLastError() == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

int npd_selftest_wait_timeout(int64_t limit_cycles, int32_t* out3, void* cuda_stream) {
  // the limit is kept short on purpose: this entry point exists to run the time-out path, not to wait
  if (out3 == nullptr || limit_cycles < 1 || limit_cycles > 100000000) return NPD_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(out3, 0, 3 * sizeof(int32_t), st) != cudaSuccess) return NPD_ECUDA;
  wait_timeout_selftest_kernel<<<1, 128, 0, st>>>(static_cast<long long>(limit_cycles), out3);
  return cudaGetLastError() == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

int npd_debug_chunk_schedule(int32_t row_blocks, int32_t d, int32_t chunk_cols, int32_t pairs, int32_t pair,
                             int32_t max_units, int32_t* units, int32_t* n_units) {
  if (row_blocks < 0 || d < 1 || chunk_cols < 1 || pairs < 1 || pair < 0 || pair >= pairs || max_units < 0 ||
      n_units == nullptr || (max_units > 0 && units == nullptr))
    return NPD_EINVAL;
  GemmParams gp{};
  chunk_problems(d, chunk_cols, false, false, gp.pr);
  gp.nprob = 2;
  GemmWalk walk;
  walk.init(gp, row_blocks, pair, pairs);
  int n = 0, prob = 0;
  GemmUnit u;
  while (walk.next(prob, u)) {
    if (n < max_units) {
      int32_t* o = units + 5 * n;
      o[0] = prob;
      o[1] = u.m0;
      o[2] = u.n0;
      o[3] = u.kt0;
      o[4] = u.kt1;
    }
    ++n;
  }
  *n_units = n;
  return NPD_OK;
}

int npd_last_status(const void* workspace, void* cuda_stream, int32_t* host_status) {
  if (workspace == nullptr || host_status == nullptr) return NPD_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(host_status, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return NPD_ECUDA;
  return cudaStreamSynchronize(st) == cudaSuccess ? NPD_OK : NPD_ECUDA;
}

// ---------------------------------------------------------------------------------------
// Forward pass for callers that cannot allocate device memory.
//
// Some users of this library cannot hand it a workspace: a plug-in running inside a host
// framework that claimed the whole device memory for its own pool at start-up (a fresh
// cudaMalloc there simply fails), or a steady-state serving/training loop that may not
// stall the device (cudaMalloc and cudaFree synchronise it).  For them the forward pass'
// scratch (the per-split softmax partials, the log-sum-exps and the status word) lives
// in the fixed array below, which is part of the library image: every GPU that loads the
// library carries these NPD_STATIC_SCRATCH_BYTES (+1 KiB) until the process exits.
//
// g_static_scratch names the array for DEVICE code.  In host code the same identifier is
// only a host-side handle, not a device address, so the real address is asked for once
// per device with cudaGetSymbolAddress (with that device current) and cached.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[NPD_STATIC_SCRATCH_BYTES + 1024];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_scratch_addr[kMaxDevices] = {};
std::mutex g_static_scratch_mutex;

// Device address of the static scratch on the current device, 1024-byte aligned.
int static_scratch_base(uint8_t** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NPD_ECUDA;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return NPD_ECUDA;
    g_static_scratch_addr[dev] = ptr;
  }
  const uintptr_t a = reinterpret_cast<uintptr_t>(g_static_scratch_addr[dev]);
  *out = reinterpret_cast<uint8_t*>((a + 1023) & ~static_cast<uintptr_t>(1023));
  return NPD_OK;
}
}  // namespace

int npd_kd_forward_noalloc(const npd_kd_args* args, void* cuda_stream, int32_t* host_status) {
  if (args == nullptr || args->size != sizeof(npd_kd_args)) return NPD_EINVAL;
  if (args->d_hidden != nullptr || args->d_weight != nullptr) return NPD_EINVAL;  // forward only
  npd_kd_args a = *args;
  a.workspace = nullptr;
  a.workspace_bytes = 0;
  size_t need = 0;
  int rc = npd_workspace_bytes(&a, &need);
  if (rc != NPD_OK) return rc;
  if (need > static_cast<size_t>(NPD_STATIC_SCRATCH_BYTES)) return NPD_EWORKSPACE;  // problem too large
  uint8_t* base = nullptr;
  if ((rc = static_scratch_base(&base)) != NPD_OK) return rc;
  a.workspace = base;
  a.workspace_bytes = NPD_STATIC_SCRATCH_BYTES;
  // npd_kd_fwd_bwd clears the status word itself and overwrites every partial it later reads,
  // so nothing of the previous call's contents survives into this one.
  if ((rc = npd_kd_fwd_bwd(&a, cuda_stream)) != NPD_OK) return rc;
  if (host_status != nullptr) return npd_last_status(base, cuda_stream, host_status);
  return NPD_OK;
}

int npd_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int64_t lda, int32_t a_mn_major,
                  const void* B, int64_t ldb, int32_t b_mn_major, void* out, int64_t ldo,
                  int32_t out_mode, int32_t k_splits, void* cuda_stream) {
  if (M < 1 || N < 1 || K < 1 || A == nullptr || B == nullptr || out == nullptr) return NPD_EINVAL;
  if (out_mode < NPD_GEMM_STORE_F32 || out_mode > NPD_GEMM_ATOMIC_F32 || k_splits < 1) return NPD_EINVAL;
  if (k_splits > 1 && out_mode != NPD_GEMM_ATOMIC_F32 && out_mode != NPD_GEMM_ADD_F32) return NPD_EINVAL;
  const bool f32 = out_mode != NPD_GEMM_STORE_BF16;
  if (!aligned16(A) || !aligned16(B) || !aligned16(out) || (lda % 8) || (ldb % 8) || (ldo % (f32 ? 4 : 8)))
    return NPD_EALIGN;
  if (lda < (a_mn_major ? M : K) || ldb < (b_mn_major ? N : K) || ldo < N) return NPD_ESHAPE;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc != NPD_OK) return rc;
  if (di.cc_major != 10) return NPD_EARCH;
  GemmProblem pr{};
  pr.M = M;
  pr.N = N;
  pr.K = K;
  pr.a_mn = a_mn_major != 0;
  pr.b_mn = b_mn_major != 0;
  pr.k_splits = k_splits;
  pr.out_f32 = f32;
  pr.out_reduce = out_mode == NPD_GEMM_ADD_F32 || out_mode == NPD_GEMM_ATOMIC_F32;
  const GemmOperands ops{A, lda, B, ldb, out, ldo};
  return launch_gemm(1, &pr, &ops, nullptr, 0, nullptr, di.sms, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
