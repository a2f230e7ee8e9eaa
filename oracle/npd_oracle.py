"""CPU oracle for the packed-sequence distillation loss step of Near-Policy Distillation.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
method computes; the CUDA library is checked against it.  Only the tests, the
smoke check and the CPU-baseline leg of the benchmark may import it.  It shares
no code, tables or helpers with the CUDA path and never imports it.

Everything is evaluated in float64 with NumPy.  The only library primitives used
as steps are ``numpy.matmul`` (the LM-head product and the two gradient
products), ``numpy.exp`` / ``numpy.log`` and reductions.  No blocking, fusion or
online rescaling: each function is the definition written out.

Notation (paper, Section 3 and Algorithm 1):
  T packed tokens, d hidden size, V vocabulary size, S segments (samples);
  H[T,d]   student hidden states entering the LM head;
  W[V,d]   LM-head weight, so the student logits are O_S = H W^T
           (Algorithm 1, "Compute Student Logits");
  O_T[T,V] teacher logits stored by the annotation phase (Algorithm 1, Phase 2);
  tau      softmax temperature of the distillation term;
  m[T]     loss mask (1 = response token, contributes), labels y[T] (<0 = none);
  cu[S+1]  packed-segment boundaries, segment s = tokens cu[s] <= t < cu[s+1].

Readings taken where the paper leaves a choice (each also listed in the design
notes): the KL support is the whole vocabulary (Eq. 2 with V_top-k = V, dense
teacher logits; a row whose teacher logit is -inf outside its top-k reproduces the
top-k form with the teacher renormalised on its support); the KL is the plain
divergence at temperature tau with no tau^2 factor; the per-sequence
cross-entropy L_theta of Eq. 3 is the token mean over the positions that carry
loss; both ends of the keep interval are inclusive (Proximal Learning Zone,
0 <= Delta <= threshold).

The composite objective follows Eq. 1 with the cross-entropy at temperature 1; the
top-k functions follow Eq. 2 as printed, with p_T the softmax of the k stored logits.

Pins: every function below is pinned by tests/test_oracle_*.py against closed
forms, finite differences, SciPy/PyTorch library routines, brute force and a
hand-worked table (tests/golden/).  The one thing that cannot be pinned is the
*distribution* of Delta-IFD over real data (the paper's zone fractions come from
a proprietary set): parity unpinned for that distribution; the rule itself is
pinned.
"""

from __future__ import annotations

import numpy as np

__all__ = [
    "student_logits",
    "log_softmax",
    "kd_token_losses",
    "kd_logit_gradient",
    "kd_backward",
    "kd_dhidden_rows",
    "kd_dweight_rows",
    "composite_token_loss",
    "composite_logit_gradient",
    "composite_backward",
    "topk_kd_token_losses",
    "topk_kd_logit_gradient",
    "topk_kd_backward",
    "validate_step_inputs",
    "validate_cu_seqlens",
    "segment_ids",
    "segment_stats",
    "reverse_kl_token",
    "ifd_scores",
    "delta_ifd_select",
    "perplexity_scores",
    "nearest_rank_percentile",
    "pack_first_fit_decreasing",
]


def _f64(x) -> np.ndarray:
    return np.asarray(x, dtype=np.float64)


# --------------------------------------------------------------------------- #
# LM head and softmax (Algorithm 1: "Compute Student Logits", "Compute Probs")
# --------------------------------------------------------------------------- #

def student_logits(H, W) -> np.ndarray:
    """O_S = H W^T, the last linear layer of the student (Algorithm 1, student
    logits step).  No bias."""
    return np.matmul(_f64(H), _f64(W).T)


def log_softmax(x) -> np.ndarray:
    """log Softmax(x) along the last axis.  -inf entries are allowed (probability
    zero); a row must hold at least one finite entry."""
    x = _f64(x)
    mx = np.max(x, axis=-1, keepdims=True)
    with np.errstate(divide="ignore"):
        lse = mx + np.log(np.sum(np.exp(x - mx), axis=-1, keepdims=True))
    return x - lse


# --------------------------------------------------------------------------- #
# Per-token losses (Eq. 2; the cross-entropy that Eq. 3 is built from)
# --------------------------------------------------------------------------- #

def kd_token_losses(H, W, teacher_logits, labels, loss_mask, tau: float):
    """Per-token distillation loss and per-token negative log-likelihoods.

    kl[t]    = m_t * sum_c p_T(c) * (log p_T(c) - log p_S(c))       (Eq. 2)
               with p_T = Softmax(O_T[t]/tau), p_S = Softmax(O_S[t]/tau)
               (Algorithm 1, "Compute Probs") and 0*log 0 = 0;
    nll_s[t] = -m_t * [y_t>=0] * log Softmax(O_S[t])[y_t]   (student CE term,
               temperature 1: the L_theta of Eq. 3 for the student);
    nll_t[t] = the same for the teacher logits O_T[t].

    Returns (kl, nll_s, nll_t), float64 arrays of length T.
    """
    H = _f64(H)
    T = H.shape[0]
    O_S = student_logits(H, W)
    O_T = _f64(teacher_logits)[:, : O_S.shape[1]]
    labels = np.asarray(labels, dtype=np.int64)
    m = np.asarray(loss_mask).astype(bool)

    logp_T = log_softmax(O_T / tau)
    logp_S = log_softmax(O_S / tau)
    p_T = np.exp(logp_T)
    with np.errstate(invalid="ignore"):
        terms = p_T * (logp_T - logp_S)
    terms = np.where(p_T > 0.0, terms, 0.0)          # 0 * log 0 = 0
    kl = np.where(m, np.sum(terms, axis=1), 0.0)

    has = m & (labels >= 0)
    y = np.where(labels >= 0, labels, 0)
    rows = np.arange(T)
    nll_s = np.where(has, -log_softmax(O_S)[rows, y], 0.0)
    nll_t = np.where(has, -log_softmax(O_T)[rows, y], 0.0)
    return kl, nll_s, nll_t


# --------------------------------------------------------------------------- #
# Gradients of L = grad_scale * sum_t m_t * kl[t]
# --------------------------------------------------------------------------- #

def kd_logit_gradient(H, W, teacher_logits, loss_mask, tau: float, grad_scale: float):
    """dL/dO_S for L = grad_scale * sum_t kl[t]:

        dO_S[t,c] = grad_scale * m_t * (p_S(c) - p_T(c)) / tau

    (derivative of Eq. 2 through Softmax(O_S/tau); the teacher is constant,
    Algorithm 1 computes its logits without gradient)."""
    O_S = student_logits(H, W)
    O_T = _f64(teacher_logits)[:, : O_S.shape[1]]
    p_S = np.exp(log_softmax(O_S / tau))
    p_T = np.exp(log_softmax(O_T / tau))
    m = np.asarray(loss_mask).astype(np.float64)[:, None]
    return grad_scale * m * (p_S - p_T) / tau


def kd_backward(H, W, teacher_logits, loss_mask, tau: float, grad_scale: float):
    """Chain rule through O_S = H W^T (Algorithm 1, "Update" step, restricted to
    the LM head):  dH = dO_S W,  dW = dO_S^T H.  Returns (dH[T,d], dW[V,d])."""
    dO = kd_logit_gradient(H, W, teacher_logits, loss_mask, tau, grad_scale)
    return np.matmul(dO, _f64(W)), np.matmul(dO.T, _f64(H))


def kd_dhidden_rows(H, W, teacher_logits, loss_mask, tau, grad_scale, token_rows):
    """Rows ``token_rows`` of dH.  A token's gradient depends on that token only,
    so this is kd_backward restricted to those tokens."""
    r = np.asarray(token_rows, dtype=np.int64)
    dO = kd_logit_gradient(_f64(H)[r], W, _f64(teacher_logits)[r],
                           np.asarray(loss_mask)[r], tau, grad_scale)
    return np.matmul(dO, _f64(W))


def kd_dweight_rows(H, W, teacher_logits, loss_mask, tau, grad_scale, vocab_rows,
                    token_group: int = 0):
    """Rows ``vocab_rows`` of dW = dO_S^T H.  Needs p_S(c), hence the full
    softmax denominator, of every token, so all T tokens are evaluated.

    dW is a sum over tokens; ``token_group`` > 0 only bounds memory by adding
    the tokens' contributions in consecutive groups of that many tokens (the
    same sum, taken in the same token order).  ``teacher_logits`` may be any
    object that yields rows by slicing (e.g. a memory-mapped or torch CPU
    tensor converted slice by slice)."""
    c = np.asarray(vocab_rows, dtype=np.int64)
    T = len(H)
    g = T if token_group <= 0 else int(token_group)
    out = np.zeros((c.size, np.shape(H)[1]))
    for t0 in range(0, T, g):
        t1 = min(T, t0 + g)
        Hg = _f64(np.asarray(H[t0:t1], dtype=np.float64))
        Zg = _f64(np.asarray(teacher_logits[t0:t1], dtype=np.float64))
        dO = kd_logit_gradient(Hg, W, Zg, np.asarray(loss_mask[t0:t1]), tau, grad_scale)
        out += np.matmul(dO[:, c].T, Hg)
    return out


# --------------------------------------------------------------------------- #
# Policy-lag monitor (appendix, "Analysis of Policy Latency")
# --------------------------------------------------------------------------- #

def reverse_kl_token(H, W, generator_logits, loss_mask, tau: float = 1.0):
    """Per-token D_KL(pi_learner || pi_generator), the quantity the appendix tracks to bound
    the policy lag:  the learner is the current student, p_L = Softmax(H W^T / tau), the
    generator's logits for the same positions are given;

        rkl[t] = m_t * sum_c p_L(c) (log p_L(c) - log p_G(c)).

    Note the direction: the learner's distribution weighs the sum (Eq. 2 has the teacher's)."""
    O_L = student_logits(H, W)
    O_G = _f64(generator_logits)[:, : O_L.shape[1]]
    logp_L = log_softmax(O_L / tau)
    logp_G = log_softmax(O_G / tau)
    p_L = np.exp(logp_L)
    with np.errstate(invalid="ignore"):
        terms = p_L * (logp_L - logp_G)
    terms = np.where(p_L > 0.0, terms, 0.0)
    m = np.asarray(loss_mask).astype(bool)
    return np.where(m, terms.sum(axis=1), 0.0)


# --------------------------------------------------------------------------- #
# Composite objective (Eq. 1): L_total = (1 - lambda) L_CE + lambda L_KD
# --------------------------------------------------------------------------- #

def composite_token_loss(kl, nll_s, lam: float):
    """Eq. 1 token by token: (1 - lam) * CE_t + lam * KD_t, with CE_t the student's
    negative log-likelihood of the label (temperature 1) and KD_t the distillation
    term of Eq. 2, both already masked."""
    return (1.0 - lam) * _f64(nll_s) + lam * _f64(kl)


def composite_logit_gradient(H, W, teacher_logits, labels, loss_mask, tau: float,
                             grad_scale: float, lam: float):
    """dL/dO_S for L = grad_scale * sum_t m_t ((1 - lam) CE_t + lam KD_t)  (Eq. 1):

        dO_S[t,c] = grad_scale * m_t * ( lam (p_S^tau(c) - p_T^tau(c)) / tau
                                         + (1 - lam) [y_t>=0] (p_S^1(c) - [c = y_t]) )

    p^tau = Softmax(./tau); the cross-entropy is taken at temperature 1."""
    O_S = student_logits(H, W)
    T, V = O_S.shape
    labels = np.asarray(labels, dtype=np.int64)
    m = np.asarray(loss_mask).astype(np.float64)[:, None]
    d_kd = kd_logit_gradient(H, W, teacher_logits, loss_mask, tau, 1.0)
    has = (labels >= 0).astype(np.float64)[:, None]
    onehot = np.zeros((T, V))
    onehot[np.arange(T)[labels >= 0], labels[labels >= 0]] = 1.0
    d_ce = m * has * (np.exp(log_softmax(O_S)) - onehot)
    return grad_scale * (lam * d_kd + (1.0 - lam) * d_ce)


def composite_backward(H, W, teacher_logits, labels, loss_mask, tau: float, grad_scale: float,
                       lam: float):
    """dH = dO_S W, dW = dO_S^T H for the composite objective (Eq. 1, Algorithm 1 "Update")."""
    dO = composite_logit_gradient(H, W, teacher_logits, labels, loss_mask, tau, grad_scale, lam)
    return np.matmul(dO, _f64(W)), np.matmul(dO.T, _f64(H))


# --------------------------------------------------------------------------- #
# Eq. 2 as printed: the teacher is stored as its k largest logits per token
# --------------------------------------------------------------------------- #

def _topk_probs(topk_values, tau):
    """p_T over the stored support: Softmax of the k stored logits / tau.  (Only the k
    logits exist, so the teacher distribution is the one they define.)"""
    return np.exp(log_softmax(_f64(topk_values) / tau))


def topk_kd_token_losses(H, W, topk_values, topk_indices, labels, loss_mask, tau: float):
    """Eq. 2 with the sum over V_top-k:

        kl[t] = m_t * sum_{j<k} p_T(j) (log p_T(j) - log p_S(idx[t,j]))

    p_T = Softmax over the k stored teacher logits (/tau), p_S = Softmax(O_S[t]/tau) over
    the whole vocabulary, evaluated at the stored indices.  Also returns the student's
    per-token cross-entropy at the labels (temperature 1), as kd_token_losses does.
    Returns (kl, nll_s)."""
    H = _f64(H)
    T = H.shape[0]
    O_S = student_logits(H, W)
    idx = np.asarray(topk_indices, dtype=np.int64)
    labels = np.asarray(labels, dtype=np.int64)
    m = np.asarray(loss_mask).astype(bool)
    p_T = _topk_probs(topk_values, tau)
    logp_T = log_softmax(_f64(topk_values) / tau)
    logp_S = np.take_along_axis(log_softmax(O_S / tau), idx, axis=1)
    with np.errstate(invalid="ignore"):
        terms = p_T * (logp_T - logp_S)
    terms = np.where(p_T > 0.0, terms, 0.0)
    kl = np.where(m, terms.sum(axis=1), 0.0)
    has = m & (labels >= 0)
    y = np.where(labels >= 0, labels, 0)
    nll_s = np.where(has, -log_softmax(O_S)[np.arange(T), y], 0.0)
    return kl, nll_s


def topk_kd_logit_gradient(H, W, topk_values, topk_indices, loss_mask, tau: float,
                           grad_scale: float):
    """dL/dO_S for L = grad_scale * sum_t kl[t] of the top-k form:

        dO_S[t,c] = grad_scale * m_t * (p_S(c) - sum_{j: idx[t,j]=c} p_T(j)) / tau

    (the stored probabilities sum to one, so the student term keeps its full weight)."""
    O_S = student_logits(H, W)
    idx = np.asarray(topk_indices, dtype=np.int64)
    p_S = np.exp(log_softmax(O_S / tau))
    p_T = _topk_probs(topk_values, tau)
    dense_T = np.zeros_like(p_S)
    np.add.at(dense_T, (np.arange(O_S.shape[0])[:, None], idx), p_T)
    m = np.asarray(loss_mask).astype(np.float64)[:, None]
    return grad_scale * m * (p_S - dense_T) / tau


def topk_kd_backward(H, W, topk_values, topk_indices, loss_mask, tau: float, grad_scale: float):
    dO = topk_kd_logit_gradient(H, W, topk_values, topk_indices, loss_mask, tau, grad_scale)
    return np.matmul(dO, _f64(W)), np.matmul(dO.T, _f64(H))


# --------------------------------------------------------------------------- #
# Packed segments (sequence packing, Algorithm 1 Phase 1) and their statistics
# --------------------------------------------------------------------------- #

def validate_step_inputs(H, teacher_logits, labels, loss_mask, V: int, topk_indices=None) -> bool:
    """What the step may assume about its inputs and does not check by default.  True iff
      * every label is below V (a label < 0 means "none"; one >= V names no class),
      * with a dense teacher: no logit of a token that carries loss is NaN or +inf, and every such
        token has at least one finite teacher logit (-inf entries only remove classes from the support
        of Eq. 2; a row that is entirely -inf has no distribution),
      * with a top-k teacher: every stored index lies in [0, V),
      * the hidden states of the tokens that carry loss are finite.
    Tokens with loss_mask 0 are never read by the step, so nothing is required of their rows."""
    m = np.asarray(loss_mask).astype(bool)
    y = np.asarray(labels, dtype=np.int64)
    if np.any(y >= V):
        return False
    if not np.all(np.isfinite(_f64(H)[m])):
        return False
    if topk_indices is not None:
        idx = np.asarray(topk_indices, dtype=np.int64)[m]
        return bool(np.all((idx >= 0) & (idx < V)))
    Z = _f64(teacher_logits)[m][:, :V]
    if np.any(np.isnan(Z)) or np.any(np.isposinf(Z)):
        return False
    return bool(np.all(np.any(np.isfinite(Z), axis=1)))


def validate_cu_seqlens(cu, T: int) -> bool:
    """True iff cu is a valid boundary list: cu[0]=0, strictly increasing,
    cu[-1]=T (every segment non-empty)."""
    cu = np.asarray(cu, dtype=np.int64)
    if cu.ndim != 1 or cu.size < 2:
        return False
    return bool(cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) > 0))


def segment_ids(cu, T: int) -> np.ndarray:
    """seg_id[t] = s with cu[s] <= t < cu[s+1]."""
    cu = np.asarray(cu, dtype=np.int64)
    out = np.empty(T, dtype=np.int32)
    for s in range(cu.size - 1):
        out[cu[s]: cu[s + 1]] = s
    return out


def segment_stats(cu, loss_mask, labels, kl, nll_s, nll_t):
    """Per-sample statistics that the Delta-IFD filter consumes.

    For each segment s (one packed sample):
      kl_sum[s]    = sum_t m_t kl[t]
      nll_s_sum[s] = sum_t m_t [y_t>=0] nll_s[t]     (numerator of L_theta, Eq. 3)
      nll_t_sum[s] = the same for the teacher
      count[s]     = sum_t m_t [y_t>=0]              (its token count, int32)
    """
    cu = np.asarray(cu, dtype=np.int64)
    S = cu.size - 1
    m = np.asarray(loss_mask).astype(bool)
    has = m & (np.asarray(labels, dtype=np.int64) >= 0)
    kl, nll_s, nll_t = _f64(kl), _f64(nll_s), _f64(nll_t)
    kl_sum = np.zeros(S)
    s_sum = np.zeros(S)
    t_sum = np.zeros(S)
    count = np.zeros(S, dtype=np.int32)
    for s in range(S):
        lo, hi = int(cu[s]), int(cu[s + 1])
        for t in range(lo, hi):
            if m[t]:
                kl_sum[s] += kl[t]
            if has[t]:
                s_sum[s] += nll_s[t]
                t_sum[s] += nll_t[t]
                count[s] += 1
    return kl_sum, s_sum, t_sum, count


# --------------------------------------------------------------------------- #
# IFD, Delta-IFD and the three-zone rule (Eq. 3, Eq. 4, Section 3.2)
# --------------------------------------------------------------------------- #

def ifd_scores(cond_seg, uncond_seg, nll_sum, count, dtype=np.float64):
    """IFD(Q,A) = L(A|Q) / L(A)  (Eq. 3) for each sample i, where L is the
    token-mean cross-entropy: L(A|Q) from segment cond_seg[i] (prompt + answer,
    prompt masked), L(A) from segment uncond_seg[i] (answer alone).

    ``dtype`` is the arithmetic type of the three operations (two means, one
    ratio); float32 reproduces a float32 evaluation operation by operation.
    A sample with an empty segment (count 0) or a zero denominator scores NaN.
    """
    f = np.dtype(dtype).type
    ci = np.asarray(cond_seg, dtype=np.int64)
    ui = np.asarray(uncond_seg, dtype=np.int64)
    nll_sum = np.asarray(nll_sum).astype(dtype)
    count = np.asarray(count)
    out = np.empty(ci.size, dtype=dtype)
    for i in range(ci.size):
        nc, nu = int(count[ci[i]]), int(count[ui[i]])
        if nc <= 0 or nu <= 0:
            out[i] = np.nan
            continue
        mean_c = f(nll_sum[ci[i]]) / f(nc)
        mean_u = f(nll_sum[ui[i]]) / f(nu)
        out[i] = mean_c / mean_u if mean_u != 0 else np.nan
    return out


def delta_ifd_select(cond_seg, uncond_seg, nll_s_sum, nll_t_sum, count,
                     lo: float, hi: float, require_teacher_ifd_le_1: bool = False,
                     dtype=np.float64, score: str = "delta", lo_inclusive: bool = True,
                     hi_inclusive: bool = True):
    """Delta_IFD = IFD_Teacher - IFD_Student  (Eq. 4) and the keep rule of the
    Proximal Learning Zone:  keep iff lo <= Delta <= hi (both ends inclusive;
    the paper's lo is 0 and hi its difficulty threshold).  Delta < lo is the
    Degenerate Zone, Delta > hi the Cognitive Disconnect Zone.  The optional
    extra condition IFD_Teacher <= 1 is the "teacher confirms base quality"
    remark of the zone description.  NaN scores are never kept.

    The filter ablation (the table of filtering metrics and selection scopes) tests the
    same interval rule on other scores and with open ends: ``score`` picks what is
    tested ("delta", "ifd_teacher" or "ifd_student"), ``lo_inclusive`` / ``hi_inclusive``
    say whether an end belongs to the scope; an infinite end leaves that side open-ended.

    Returns (ifd_teacher, ifd_student, delta, keep uint8, n_keep int).
    """
    ifd_t = ifd_scores(cond_seg, uncond_seg, nll_t_sum, count, dtype)
    ifd_s = ifd_scores(cond_seg, uncond_seg, nll_s_sum, count, dtype)
    delta = (ifd_t - ifd_s).astype(dtype)
    f = np.dtype(dtype).type
    tested = {"delta": delta, "ifd_teacher": ifd_t, "ifd_student": ifd_s}[score]
    with np.errstate(invalid="ignore"):
        above = (tested >= f(lo)) if lo_inclusive else (tested > f(lo))
        below = (tested <= f(hi)) if hi_inclusive else (tested < f(hi))
        keep = above & below
        if require_teacher_ifd_le_1:
            keep &= ifd_t <= f(1.0)
    keep &= ~np.isnan(tested)
    return ifd_t, ifd_s, delta, keep.astype(np.uint8), int(keep.sum())


def perplexity_scores(seg, nll_sum, count, dtype=np.float64):
    """Per-sample perplexity, the classical filtering metric of the filter ablation (table of
    filtering metrics, row "Perplexity (PPL)"):

        PPL_i = exp( nll_sum[seg_i] / count[seg_i] ),

    the exponential of the token-mean cross-entropy of the sample's answer tokens (the same
    per-sequence loss L_theta that Eq. 3 divides), i.e. the inverse geometric mean of the
    probabilities the model gives the answer tokens.  A sample without such tokens scores NaN.
    The paper lists the metric with the scope "Weighted" and does not say how the weight enters
    training, so only the score is defined here.  ``dtype`` is the arithmetic type of the two
    operations (one mean, one exponential)."""
    f = np.dtype(dtype).type
    si = np.asarray(seg, dtype=np.int64)
    nll_sum = np.asarray(nll_sum).astype(dtype)
    count = np.asarray(count)
    out = np.empty(si.size, dtype=dtype)
    for i in range(si.size):
        n = int(count[si[i]])
        out[i] = np.exp(f(nll_sum[si[i]]) / f(n)) if n > 0 else np.nan
    return out


def nearest_rank_percentile(values, q: float) -> float:
    """Nearest-rank percentile of the finite entries: sort ascending and take
    element ceil(q*n)-1.  Used only to turn "threshold at the 80th percentile"
    of a workload description into a number passed to both sides."""
    v = np.sort(_f64(values)[np.isfinite(_f64(values))])
    if v.size == 0:
        return float("nan")
    k = int(np.ceil(q * v.size)) - 1
    return float(v[min(max(k, 0), v.size - 1)])


# --------------------------------------------------------------------------- #
# Sequence packing (Algorithm 1, Phase 1: S_pack <- Pack(D_select, Length = L))
# --------------------------------------------------------------------------- #

def pack_first_fit_decreasing(lengths, keep, capacity: int):
    """Packs the kept samples into rows of at most ``capacity`` tokens.

    The paper names the step but not the algorithm; the reading taken is first-fit
    decreasing: the kept samples are visited from the longest to the shortest (ties: lower
    sample index first) and each goes into the first row, in order of creation, that still
    has room; if none has, a new row is opened.  A sample longer than the capacity is cut to
    the capacity (a row is a fixed-length sequence).  Samples of length 0 are dropped.

    Returns (order, row_of, cu_seqlens, row_ptr):
      order[j]      sample placed j-th in the packed stream (rows back to back, samples
                    within a row in the order they were placed),
      row_of[j]     its row,
      cu_seqlens    [len(order)+1] token boundaries of the packed stream,
      row_ptr       [rows+1] index into ``order`` where each row starts.
    """
    lengths = np.asarray(lengths, dtype=np.int64)
    keep = np.ones(lengths.size, dtype=bool) if keep is None else np.asarray(keep).astype(bool)
    cand = [i for i in range(lengths.size) if keep[i] and lengths[i] > 0]
    cand.sort(key=lambda i: (-min(int(lengths[i]), capacity), i))
    rows, room = [], []
    for i in cand:
        n = min(int(lengths[i]), capacity)
        for r in range(len(rows)):
            if room[r] >= n:
                rows[r].append(i)
                room[r] -= n
                break
        else:
            rows.append([i])
            room.append(capacity - n)
    order = [i for r in rows for i in r]
    row_of = [r for r, members in enumerate(rows) for _ in members]
    cu = np.concatenate([[0], np.cumsum([min(int(lengths[i]), capacity) for i in order])]).astype(np.int32)
    row_ptr = np.concatenate([[0], np.cumsum([len(m) for m in rows])]).astype(np.int32)
    return (np.asarray(order, dtype=np.int32), np.asarray(row_of, dtype=np.int32), cu, row_ptr)
