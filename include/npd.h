/*
 * npd.h - C ABI of the packed-sequence distillation loss step of Near-Policy
 * Distillation (NPD), implemented as hand-written CUDA kernels for NVIDIA B200
 * (sm_100a).
 *
 * What the library computes (paper notation; T packed tokens, d hidden size,
 * V vocabulary, S packed segments, tau softmax temperature):
 *
 *   O_S = H W^T                         Algorithm 1, "Compute Student Logits"
 *                                       (LM head only; the transformer body is
 *                                       the caller's)
 *   p_T = Softmax(O_T / tau),           Algorithm 1, "Compute Probs"
 *   p_S = Softmax(O_S / tau)
 *   kl[t]  = m_t * sum_c p_T(c) log(p_T(c)/p_S(c))          Eq. 2, with the
 *            support taken as the whole vocabulary (dense teacher logits; an
 *            entry of -inf removes a class from the support)
 *   nll_student[t] = -m_t [y_t>=0] log Softmax(O_S[t])[y_t]   cross-entropy
 *   nll_teacher[t] = -m_t [y_t>=0] log Softmax(O_T[t])[y_t]   behind Eq. 3
 *   dO_S[t,c] = grad_scale * m_t * (p_S(c) - p_T(c)) / tau    gradient of Eq. 2
 *   dH = dO_S W,   dW = dO_S^T H                              Algorithm 1, "Update"
 *   per-segment sums and counts over cu_seqlens               inputs of Eq. 3
 *   IFD = L(A|Q)/L(A) (Eq. 3), Delta = IFD_T - IFD_S (Eq. 4),
 *   keep = lo <= Delta <= hi (Proximal Learning Zone, Section 3.2)
 *
 * Options: the composite objective of Eq. 1 (cross-entropy term added to the gradient,
 * NPD_KD_COMPOSITE_LOSS), the teacher stored as its k largest logits per token (Eq. 2 as
 * printed, topk_values / topk_indices), fp32 teacher logits, the learner-to-generator KL
 * of the policy-lag analysis (NPD_KD_REVERSE_KL), the selection scopes of the filter
 * ablation (flags of npd_select), and the sequence packer of Algorithm 1
 * (npd_pack_sequences).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the comment says HOST.
 *   - The caller owns every buffer.  The library allocates no device memory,
 *     keeps no problem state between calls and only enqueues work on the given stream
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *     Results are ready when the stream has been synchronised.  The exceptions are spelled out
 *     where they are declared: npd_kd_forward_noalloc works in a fixed array inside the library
 *     image, and two per-thread diagnostic counters (npd_last_launch_count,
 *     npd_last_copy_bytes) remember the last call for benchmarks.
 *   - Return value: NPD_OK (0) or a negative npd_status.  Argument errors are
 *     found on the host before anything is launched.  Errors found on the device
 *     (malformed cu_seqlens, a bounded wait that ran out) are recorded in the
 *     workspace and read with npd_last_status().
 *   - No exceptions, no abort(), no device traps.  Every device-side wait on an mbarrier is
 *     bounded (about 2 s of SM clocks).  When one runs out the CTA raises an abort flag that all
 *     its roles poll; warps that meet at named barriers decide together, through a vote at
 *     such a barrier, whether to go on, so none is left waiting alone; producers give the copies
 *     they have issued a last bounded grace period to land; both CTAs of a pair meet at the closing
 *     cluster barrier, tensor memory is freed and the status word reads NPD_ETIMEOUT.
 *   - Needs a device of compute capability 10.x; otherwise NPD_EARCH.
 */
#ifndef NPD_H_
#define NPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum npd_status {
  NPD_OK = 0,
  NPD_EINVAL = -1,      /* null pointer, bad size field, non-positive dimension, tau <= 0 */
  NPD_ESHAPE = -2,      /* d not a multiple of 64, a row stride smaller than the row, S > T */
  NPD_EALIGN = -3,      /* a base pointer or row stride of a tensor operand not 16-byte aligned */
  NPD_ESEQ = -4,        /* cu_seqlens malformed (found on the device) */
  NPD_EARCH = -5,       /* current device is not compute capability 10.x */
  NPD_EWORKSPACE = -6,  /* workspace NULL, misaligned or smaller than npd_workspace_bytes() */
  NPD_ECUDA = -7,       /* a CUDA runtime or driver call failed */
  NPD_ETIMEOUT = -8,    /* a bounded device-side wait expired (found on the device) */
  NPD_EUNSUPPORTED = -9,/* a documented option that this build does not implement */
  NPD_EDATA = -10       /* NPD_KD_DEBUG_CHECKS found an input the step may not be given (found on the device) */
} npd_status;

enum { NPD_DTYPE_BF16 = 0, NPD_DTYPE_F32 = 1 };

/* flags of npd_kd_args */
enum {
  NPD_KD_ACCUMULATE_DW = 1, /* add into d_weight instead of overwriting it (f32 d_weight only) */
  NPD_KD_COMPOSITE_LOSS = 2,/* gradients of the composite objective of Eq. 1,
                               L_total = (1 - lambda) L_CE + lambda L_KD with lambda = kd_lambda:
                                 dO_S[t,c] = grad_scale * m_t * ( lambda (p_S - p_T) / tau
                                             + (1 - lambda) [y_t>=0] (Softmax(O_S[t])[c] - [c = y_t]) )
                               (cross-entropy at temperature 1).  Needs labels.  The per-token
                               outputs are unchanged: the loss value of a token is
                               (1 - lambda) * nll_student[t] + lambda * kl[t].  Without the flag
                               the gradients are those of Eq. 2 alone (lambda = 1). */
  NPD_KD_REVERSE_KL = 4,    /* forward only (d_hidden, d_weight NULL; dense `teacher`): kl[t] becomes
                               m_t * D_KL(p_S || p_G) = sum_c p_S(c) (log p_S(c) - log p_G(c)) with
                               p_G = Softmax(teacher[t]/tau), i.e. the divergence of the current
                               learner from the logits of the policy that generated the data, which
                               the paper's appendix tracks as policy lag.  Needs finite logits. */
  NPD_KD_DEBUG_CHECKS = 16, /* before anything else, check on the device what the kernels otherwise take on
                               trust and record NPD_EDATA in the status word if it does not hold: every
                               label below V; for every token that carries loss finite hidden states,
                               and either (dense teacher) no NaN or +inf logit and at least one finite
                               one - a row that is entirely -inf has no distribution - or (top-k
                               teacher) every stored index inside [0, V).  Rows of tokens without loss
                               are not read.  The step runs all the same; with NPD_EDATA its outputs are
                               undefined.  Costs one more pass over the teacher logits. */
  NPD_KD_SERIALIZE_LAUNCHES = 8 /* launch every kernel fully serialised.  By default the tensor-core
                               kernels of a call are chained as programmatic dependent launches:
                               the blocks of the next kernel are scheduled, and set up their
                               barriers and tensor memory, while the last blocks of the kernel
                               before it are still running, and wait for its completion before
                               they read or write anything it touches.  Same results either way;
                               the flag is for debugging and for timing comparisons. */
};

/*
 * Arguments of the fused KD forward+backward (Algorithm 1, Phase 3, lines
 * "Compute Student Logits" to "Update", restricted to the LM head and Eq. 2).
 *
 * Layouts are row-major with explicit row strides in ELEMENTS.  hidden, weight,
 * teacher, d_hidden and d_weight must be 16-byte aligned with row strides that
 * are multiples of 16 bytes (8 bf16 elements).  d must be a multiple of 64.
 * Any T >= 1, V >= 1 is accepted (ragged tiles are masked in the kernels).
 */
typedef struct npd_kd_args {
  size_t size;               /* = sizeof(npd_kd_args); checked */
  int32_t T, d, V, S;
  const void* hidden;        /* bf16 [T, ldh]   H                                  */
  const void* weight;        /* bf16 [V, ldw]   W (LM head, no bias)               */
  const void* teacher;       /* bf16 (or f32) [T, ldt]   O_T, ldt >= V; columns >= V ignored
                                (not read when topk > 0, see the end of the struct) */
  int64_t ldh, ldw, ldt;
  int32_t teacher_dtype;     /* NPD_DTYPE_BF16, or NPD_DTYPE_F32 (then teacher is f32
                                [T, ldt] with ldt a multiple of 4)                   */
  int32_t reserved0;
  const int32_t* cu_seqlens; /* [S+1] cu[0]=0, strictly increasing, cu[S]=T; may be NULL
                                (then S is ignored and nothing is validated)       */
  const uint8_t* loss_mask;  /* [T] 1 = token carries loss; NULL = all ones         */
  const int32_t* labels;     /* [T] class the position must predict, <0 = none;
                                NULL = no NLL outputs                              */
  float temperature;         /* tau > 0                                             */
  float grad_scale;          /* dL/d(sum_t kl[t]); e.g. 1/n_loss                    */
  /* outputs (each may be NULL unless noted) */
  float* kl;                 /* [T] required                                        */
  float* nll_student;        /* [T]                                                 */
  float* nll_teacher;        /* [T]                                                 */
  void* d_hidden;            /* bf16 [T, ldh]; NULL (with d_weight NULL) = forward only */
  void* d_weight;            /* bf16 or f32 [V, ldw]; both gradients or neither     */
  int32_t d_weight_dtype;    /* NPD_DTYPE_BF16 or NPD_DTYPE_F32                     */
  int32_t flags;
  int32_t grad_chunk_cols;   /* vocabulary columns of logit-gradient tiles that may be in
                                flight between the gradient kernel and the two
                                contractions; 0 = library default.  Bounds the scratch. */
  float kd_lambda;           /* lambda of Eq. 1 in [0,1]; read only with NPD_KD_COMPOSITE_LOSS
                                (the paper trains with 0.9) */
  void* workspace;           /* >= npd_workspace_bytes(), 1024-byte aligned         */
  size_t workspace_bytes;
  /* Optional timing hooks.  HOST array of n_phase_events cudaEvent_t (as void*), or NULL.
     Event 0 is recorded on the stream before the first kernel, event i after the i-th
     launch group, in this order: forward tiles, per-token merge, then for every
     vocabulary chunk: gradient tiles, the dW and dH contractions (one launch); last the
     dH conversion if there is one.  Groups beyond n_phase_events - 1 are not recorded.
     npd_phase_count() tells how many groups a call has. */
  void* const* phase_events;
  int32_t n_phase_events;
  int32_t reserved2;
  /* Teacher stored as its largest logits per token (Eq. 2 as printed: the sum runs over
     V_top-k).  With topk > 0 the dense `teacher` is not read (may be NULL) and
       p_T      = Softmax(topk_values[t, :] / tau) over the topk stored logits,
       kl[t]    = m_t * sum_j p_T(j) (log p_T(j) - log p_S(topk_indices[t,j])),
       dO_S[t,c] = grad_scale * m_t * lambda * (p_S(c) - sum_{j: idx[t,j]=c} p_T(j)) / tau,
     p_S still the softmax over the whole vocabulary.  nll_teacher must be NULL (the stored
     logits do not define the teacher's probability of an arbitrary label).  A stored logit
     of -inf marks an unused entry.  topk <= 16; indices must lie in [0, V). */
  const float* topk_values;    /* f32 [T, topk] */
  const int32_t* topk_indices; /* [T, topk]     */
  int32_t topk;                /* 0 = dense teacher */
  int32_t reserved3;
} npd_kd_args;

/* HOST.  Bytes of workspace npd_kd_fwd_bwd needs for these arguments (pointers
 * inside args are not read).  Depends on T, d, V, grad_chunk_cols, on whether
 * gradients are requested and on the device's SM count. */
int npd_workspace_bytes(const npd_kd_args* args, size_t* out_bytes);

/* HOST.  Number of launch groups (see phase_events) npd_kd_fwd_bwd runs for these arguments,
 * and in *out_chunks (may be NULL) the number of vocabulary chunks of the backward. */
int npd_phase_count(const npd_kd_args* args, int32_t* out_groups, int32_t* out_chunks);

/* Fused forward + backward of the distillation term (see the struct).  `args`
 * is a HOST struct holding device pointers.  Enqueues on `cuda_stream`.
 *
 * Tokens with loss_mask 0 have kl = nll = 0 and no gradient by definition; the kernels
 * compact the tokens that carry loss (on the device, from loss_mask) and spend no work
 * on the rest, so a batch with 30 % masked prompt tokens costs 30 % less.  Every output
 * element is written all the same (zeros where nothing is computed).
 *
 * The call makes no synchronising CUDA call; it can be recorded by a stream capture and
 * replayed as a CUDA graph (the tensor maps in the launch arguments bake in the buffer
 * addresses of the captured call).
 *
 * kl, nll_*, and d_weight are bitwise reproducible from run to run.  d_hidden is summed
 * over vocabulary chunks with fp32 atomic adds whose order is not fixed: a few of its
 * bf16 elements may round differently between runs. */
int npd_kd_fwd_bwd(const npd_kd_args* args, void* cuda_stream);

/*
 * Same computation from HOST buffers, for callers whose step inputs arrive in
 * host memory.  `host` and `dev` describe the same problem: `dev` is a complete,
 * valid npd_kd_args of device buffers (used as staging), `host` holds HOST
 * pointers for the per-step inputs (hidden, teacher, cu_seqlens, loss_mask,
 * labels; pinned memory for overlap) and for the per-token outputs (kl,
 * nll_student, nll_teacher).  The weight is a resident parameter and the two
 * gradients stay on the device: host->weight, d_hidden, d_weight are ignored.
 * The call copies the inputs in, runs npd_kd_fwd_bwd(dev) and copies the
 * per-token outputs back, all asynchronously on `cuda_stream`.  Of hidden and teacher
 * (or the top-k arrays) only the rows of tokens with loss_mask != 0 are copied (the host
 * mask is read during the call): the kernels never read the other rows, and the staging
 * buffers keep whatever they held there.
 */
int npd_kd_fwd_bwd_host(const npd_kd_args* host, const npd_kd_args* dev, void* cuda_stream);

/*
 * The same with the copies in on a stream of their own.  The copies wait for everything
 * queued so far on `cuda_stream` (the last user of the staging buffers in `dev`), the kernels
 * wait for the copies; the copies back run on `cuda_stream`.  A caller that alternates between
 * two sets of staging buffers, each with its own `cuda_stream`, and gives every call the same
 * `copy_stream`, gets the copies of step i+1 under the kernels of step i, one transfer at a
 * time on the link.  Creates and releases two CUDA events per call (no device memory).
 */
int npd_kd_fwd_bwd_host_streams(const npd_kd_args* host, const npd_kd_args* dev, void* copy_stream,
                                void* cuda_stream);

/*
 * Per-sample statistics for the Delta-IFD filter (the sums behind Eq. 3):
 *   kl_sum[s]    = sum_{t in s} m_t kl[t]
 *   nll_s_sum[s] = sum_{t in s} m_t [y_t>=0] nll_student[t]     (same for teacher)
 *   count[s]     = sum_{t in s} m_t [y_t>=0]                    (bit-exact)
 *   seg_id[t]    = s with cu[s] <= t < cu[s+1]                  (optional)
 * Sums are taken in fp32 in a fixed order (deterministic).  kl / nll_* / the
 * three sum outputs may be NULL in matching pairs.  loss_mask NULL = all ones,
 * labels NULL = every label valid.  `status` (int32[1], may be NULL) receives
 * NPD_ESEQ if cu_seqlens is malformed, else is left untouched.
 */
int npd_segment_stats(int32_t T, int32_t S, const int32_t* cu_seqlens,
                      const uint8_t* loss_mask, const int32_t* labels,
                      const float* kl, const float* nll_student, const float* nll_teacher,
                      float* kl_sum, float* nll_s_sum, float* nll_t_sum,
                      int32_t* count, int32_t* seg_id, int32_t* status, void* cuda_stream);

/* flags of npd_select */
enum {
  NPD_SELECT_TEACHER_IFD_LE_1 = 1,  /* also require IFD_Teacher <= 1 (Section 3.2, zone text) */
  /* the selection scopes of the paper's filter ablation: the interval tests another score,
     or has open ends (an infinite lo / hi leaves that side unbounded) */
  NPD_SELECT_SCORE_IFD_TEACHER = 2, /* keep = lo <= ifd_teacher <= hi */
  NPD_SELECT_SCORE_IFD_STUDENT = 4, /* keep = lo <= ifd_student <= hi */
  NPD_SELECT_LO_EXCLUSIVE = 8,      /* lo <  score */
  NPD_SELECT_HI_EXCLUSIVE = 16      /* score <  hi */
};

/*
 * Delta-IFD score and selection (Eq. 3, Eq. 4, three-zone rule of Section 3.2).
 * Sample i is described by two segments: cond_seg[i] holds prompt+answer with the
 * prompt masked (L(A|Q)), uncond_seg[i] the answer alone (L(A)).  With
 * L = nll_sum / count (token mean), in fp32 with IEEE division:
 *   ifd_X[i] = L_X(cond) / L_X(uncond),  X in {teacher, student}
 *   delta[i] = ifd_teacher[i] - ifd_student[i]
 *   keep[i]  = lo <= delta[i] <= hi   (both inclusive; NaN never kept)
 * A sample with an empty segment (count 0) or a zero denominator scores NaN.
 * n_keep[0] = number of kept samples.  ifd_* and delta may be NULL.
 */
int npd_select(int32_t N, const int32_t* cond_seg, const int32_t* uncond_seg,
               const float* nll_s_sum, const float* nll_t_sum, const int32_t* count,
               int32_t S, float lo, float hi, int32_t flags,
               float* ifd_teacher, float* ifd_student, float* delta,
               uint8_t* keep, int32_t* n_keep, void* cuda_stream);

/*
 * HOST (all pointers are HOST pointers; no GPU work).  Sequence packing of Algorithm 1,
 * Phase 1: S_pack <- Pack(D_select, Length = capacity).  The paper names the step, not the
 * algorithm; this is first-fit decreasing: kept samples (keep[i] != 0, or all if keep is NULL)
 * with length > 0 are visited from the longest to the shortest (ties: lower index first) and
 * put into the first row, in order of creation, with enough room, else into a new row.  A
 * sample longer than `capacity` is cut to `capacity`.
 *   order[j]      sample placed j-th in the packed stream (rows back to back)      [<= N]
 *   row_of[j]     its row                                                          [<= N]
 *   cu_seqlens    token boundaries of the packed stream, ready for npd_kd_args     [<= N+1]
 *   row_ptr       index into order where each row starts, row_ptr[rows] = placed   [<= N+1]
 *   n_placed, n_rows   how many samples were placed and how many rows were opened
 * Output arrays must hold N (resp. N+1) entries.  NPD_EINVAL on NULL outputs, N < 0 or
 * capacity < 1.  Cost O(N log N + N * rows).
 */
int npd_pack_sequences(int32_t N, const int32_t* lengths, const uint8_t* keep, int32_t capacity,
                       int32_t* order, int32_t* row_of, int32_t* cu_seqlens, int32_t* row_ptr,
                       int32_t* n_placed, int32_t* n_rows);

/*
 * Per-sample perplexity, the classical filtering metric that the paper's filter ablation (table
 * of filtering metrics and selection scopes, row "Perplexity (PPL)") compares Delta-IFD with:
 *   ppl_X[i] = exp( nll_X_sum[seg[i]] / count[seg[i]] ),   X in {student, teacher},
 * the exponential of the token-mean cross-entropy of the answer tokens of segment seg[i] (the
 * per-sequence loss of Eq. 3), in fp32 with IEEE division.  NaN for a sample without such tokens
 * (count 0) or a segment index outside [0, S).  The paper applies the metric as a weight
 * ("Weighted" scope) without saying how; only the score is computed here.  Either output (with
 * its sum array) may be NULL, not both.
 */
int npd_perplexity(int32_t N, const int32_t* seg, const float* nll_s_sum, const float* nll_t_sum,
                   const int32_t* count, int32_t S, float* ppl_student, float* ppl_teacher,
                   void* cuda_stream);

/*
 * Self-test of the time-out path (no counterpart in the paper; the failure-handling code of the
 * tensor kernels would otherwise never run on a healthy device).  Launches one small CTA that
 * waits, with the same bounded wait and the same group vote the tensor kernels use, on a barrier
 * nothing arrives on, for `limit_cycles` SM clock cycles (1 .. 1e8; a millisecond is about 2e6).
 * out3 (DEVICE, int32[3], cleared by the call): [0] the status word, NPD_ETIMEOUT afterwards;
 * [1] 1 if every thread's wait gave up; [2] cycles thread 0 spent waiting.  No copy or MMA is in
 * flight in that kernel and it always terminates.
 */
int npd_selftest_wait_timeout(int64_t limit_cycles, int32_t* out3, void* cuda_stream);

/*
 * HOST, diagnostic (no GPU work; no counterpart in the paper).  The units of work CTA pair
 * `pair` of `pairs` takes in the launch that holds the two backward contractions of one
 * vocabulary chunk (dW rows of the chunk, and the chunk's contribution to dH): the same
 * scheduling code the kernel runs, evaluated on the host so that its index arithmetic can be
 * checked without a device.  row_blocks = blocks of 128 compact rows, d = hidden size,
 * chunk_cols = vocabulary columns of the chunk.  units (HOST, int32[max_units][5]) receives
 * {problem (0 = dW, 1 = dH), first row, first column, first k-step, end k-step} per unit, in the
 * order the pair works through them; *n_units the number of units (also when it exceeds
 * max_units).
 */
int npd_debug_chunk_schedule(int32_t row_blocks, int32_t d, int32_t chunk_cols, int32_t pairs,
                             int32_t pair, int32_t max_units, int32_t* units, int32_t* n_units);

/* Synchronises `cuda_stream`, then reads the device-side status word of a
 * workspace that npd_kd_fwd_bwd used into *host_status (HOST): NPD_OK,
 * NPD_ESEQ, NPD_ETIMEOUT or (debug checks) NPD_EDATA.  Returns NPD_ECUDA if the stream itself failed. */
int npd_last_status(const void* workspace, void* cuda_stream, int32_t* host_status);

/* HOST.  Static description of a status code. */
const char* npd_strerror(int status);

/* HOST, diagnostic.  Number of kernel launches the last npd_kd_fwd_bwd call on this thread
 * enqueued (for launch accounting in benchmarks).  One of the two pieces of per-thread state
 * the library keeps; it influences nothing. */
int npd_last_launch_count(void);

/* HOST, diagnostic.  Bytes the last npd_kd_fwd_bwd_host call on this thread copied
 * host-to-device and device-to-host (per-thread state like the launch count). */
int npd_last_copy_bytes(int64_t* h2d_bytes, int64_t* d2h_bytes);

/*
 * Forward pass without any workspace from the caller.  (The paper has no counterpart
 * to this entry point; it exists for deployment.)
 *
 * For callers that cannot allocate device memory: code running inside a host framework
 * that took the whole device memory for its own pool at start-up, so that a fresh
 * cudaMalloc fails, and steady-state loops that may not stall the device, which
 * cudaMalloc and cudaFree do.  The scratch of the forward pass (softmax partials per
 * vocabulary split, per-token log-sum-exps, status word) lives in a fixed array inside
 * the library image instead: NPD_STATIC_SCRATCH_BYTES (+1 KiB) on every GPU that loads
 * the library, held until the process exits.
 *
 * `args` as for npd_kd_fwd_bwd, forward only: d_hidden and d_weight must be NULL
 * (NPD_EINVAL otherwise); workspace / workspace_bytes are ignored.  The caller still
 * passes all inputs and the kl / nll_* outputs.  A problem whose scratch
 * (npd_workspace_bytes of the same forward-only arguments) exceeds
 * NPD_STATIC_SCRATCH_BYTES is refused with NPD_EWORKSPACE before anything is launched;
 * c2's forward (T=8192, d=1536, V=151,936) needs about 40 MB.  The call makes no cudaMalloc,
 * cudaFree or other allocating call.
 *
 * The first call on each device looks up the array's device address (with that device
 * current) and caches it; make that first call outside any stream capture.  The cached address
 * does not survive a cudaDeviceReset of that device: do not use this entry point after one.  All calls on
 * a device share the one array and it keeps the previous call's contents: the library
 * clears the status word at the start of every call and overwrites every partial before
 * reading it, but two calls whose kernels overlap on the GPU (different streams, or
 * different host threads) race on it - serialise them.
 *
 * host_status (HOST, may be NULL): if given, the call synchronises `cuda_stream` and
 * stores the device-side status (NPD_OK, NPD_ESEQ, NPD_ETIMEOUT) there, as
 * npd_last_status would; if NULL the call only enqueues.
 */
#define NPD_STATIC_SCRATCH_BYTES (48u * 1024u * 1024u)
int npd_kd_forward_noalloc(const npd_kd_args* args, void* cuda_stream, int32_t* host_status);

/* out_mode of npd_gemm_bf16 */
enum {
  NPD_GEMM_STORE_F32 = 0,  /* D = acc                                                  */
  NPD_GEMM_ADD_F32 = 1,    /* D += acc, element-wise atomic adds (D must be initialised) */
  NPD_GEMM_STORE_BF16 = 2, /* D = bf16(acc)                                            */
  NPD_GEMM_ATOMIC_F32 = 3  /* same as NPD_GEMM_ADD_F32; the mode split-K is meant for   */
};

/*
 * The tensor-core contraction behind the two backward products (dH = dO_S W and
 * dW = dO_S^T H, the chain rule through Algorithm 1's student-logit step),
 * exposed as a building block:
 *     D[M,N] (+)= sum_k A[m,k] * B[n,k]      bf16 inputs, fp32 accumulation.
 * An operand is K-major (memory [rows][K], x_mn_major = 0, ld >= K) or MN-major
 * (memory [K][rows], x_mn_major = 1, ld >= rows).  Pointers 16-byte aligned, row
 * strides multiples of 16 bytes.  k_splits > 1 needs one of the two adding modes;
 * the order of the additions, and so the last bits of the sums, can differ from
 * run to run.
 */
int npd_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int64_t lda, int32_t a_mn_major,
                  const void* B, int64_t ldb, int32_t b_mn_major, void* out, int64_t ldo,
                  int32_t out_mode, int32_t k_splits, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* NPD_H_ */
