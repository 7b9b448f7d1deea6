"""Oracle attention paths in float64 numpy (test infrastructure only).

Tensors are numpy arrays laid out [B, H, N, d]: q [B,Hq,N,dqk], k [B,Hkv,N,dqk],
v [B,Hkv,N,dv], dO [B,Hq,N,dv]; query head h reads KV head h // (Hq // Hkv)
(native GQA, K/V never repeated).  ``causal`` keeps keys j <= i.

Three operand precisions share one statement of the path:

  "none"   nothing is quantised: softmax attention and its gradient exactly as
           in the paper's Section 2.3 (S=QK^T*scale, P=softmax(S), O=PV,
           dV=P^T dO, dP=dO V^T, dS=P*(dP-delta), dQ=dS K*scale, dK=dS^T Q*scale).
  "mxfp8"  every matmul operand is replaced by its E4M3 x E8M0 value, in
           blocks of 32 along that matmul's contraction dimension; products
           accumulate exactly (float64 stands for FP32 accumulation).
  "bf16"   every matmul operand is rounded to BF16 instead (no scales).

The row correction follows the paper's Section 3.3: "matched" is
delta_i = sum_j P_ij dP^_ij (Eq. 4) with P the unquantised probabilities
rebuilt from the saved LSE and dP^ the product of the quantised dO and V the
gradient pass consumes; "stale" is the saved-output shortcut
sum_k dO_ik O_ik from BF16 dO and the saved BF16 O (Section 3.2).
"""
import numpy as np

from . import mxfp8

LOG2E = 1.4426950408889634
LN2 = 0.6931471805599453


def _fq(x, axis, prec):
    """Operand as the matmul sees it: blocks of 32 along ``axis`` for mxfp8."""
    if prec == "mxfp8":
        return mxfp8.fake_quant(x, axis)
    if prec == "bf16":
        return mxfp8.round_bf16(x)
    if prec == "none":
        return np.asarray(x, dtype=np.float64)
    raise ValueError(prec)


def _future_mask(rows, n_keys):
    """True where key j lies in the future of query row i (masked out)."""
    return np.arange(n_keys)[None, :] > np.asarray(rows)[:, None]


# ----------------------------------------------------------------------------
# Reference path: Section 2.3, nothing quantised.
# ----------------------------------------------------------------------------

def ref_forward(q, k, v, scale, causal):
    """O = softmax(scale * Q K^T) V and LSE_i = log sum_j exp(S_ij)."""
    B, Hq, N, _ = q.shape
    G = Hq // k.shape[1]
    O = np.zeros((B, Hq, N, v.shape[-1]))
    LSE = np.zeros((B, Hq, N))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            S = scale * (q[b, h].astype(np.float64) @ k[b, g].astype(np.float64).T)
            if causal:
                S = np.where(_future_mask(np.arange(N), N), -np.inf, S)
            m = S.max(axis=-1)
            e = np.exp(S - m[:, None])
            l = e.sum(axis=-1)
            O[b, h] = (e / l[:, None]) @ v[b, g].astype(np.float64)
            LSE[b, h] = m + np.log(l)
    return O, LSE


def ref_backward(q, k, v, dO, scale, causal, return_internals=False):
    """Gradients of Section 2.3 with delta_i = sum_j P_ij dP_ij; dK, dV summed
    over the query heads of each KV group."""
    B, Hq, N, _ = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    dQ = np.zeros(q.shape)
    dK = np.zeros(k.shape)
    dV = np.zeros(v.shape)
    D = np.zeros((B, Hq, N))
    internals = {}
    for b in range(B):
        for h in range(Hq):
            g = h // G
            Q, K, V = (x.astype(np.float64) for x in (q[b, h], k[b, g], v[b, g]))
            dOh = dO[b, h].astype(np.float64)
            S = scale * (Q @ K.T)
            if causal:
                S = np.where(_future_mask(np.arange(N), N), -np.inf, S)
            m = S.max(axis=-1, keepdims=True)
            e = np.exp(S - m)
            P = e / e.sum(axis=-1, keepdims=True)
            dP = dOh @ V.T
            delta = (P * dP).sum(axis=-1)
            dS = P * (dP - delta[:, None])
            dV[b, g] += P.T @ dOh
            dQ[b, h] = scale * (dS @ K)
            dK[b, g] += scale * (dS.T @ Q)
            D[b, h] = delta
            if return_internals:
                internals[(b, h)] = dict(P=P, dP=dP, dS=dS)
    if return_internals:
        return dQ, dK, dV, D, internals
    return dQ, dK, dV, D


# ----------------------------------------------------------------------------
# Emulated low-precision path.
# ----------------------------------------------------------------------------

def emu_forward(q, k, v, scale, causal, prec="mxfp8", exact_stats=False, rows=None,
                max_shift=0, return_internals=False):
    """Forward with quantised matmul operands.

    Per head: S = scale * Q^ K^^T from the row-blocked copies of Q and K;
    s2 = S*log2(e); M_i = ceil(max_j s2_ij) + max_shift (an integer);
    p~_ij = 2**(s2_ij - M_i), future keys 0; l_i = sum_j p~_ij from the
    UNquantised p~ (the paper's forward: the normaliser uses the exponentials
    before the FP8 cast); LSE_i = (M_i + log2 l_i) ln 2, stored FP32;
    P^ = p~ quantised per row in aligned 32-key blocks; O = (P^ V^c) / l with V^c
    the copy of V blocked along keys; O stored BF16.

    Because the block quantiser is invariant under multiplying a block by a
    power of two (only the scale byte moves), any integer M_i gives the same P^
    values; ``max_shift`` exists so that a test can show it.

    ``exact_stats`` keeps LSE in float64 (for self-checks); ``rows`` restricts
    the computation to some query rows (each row is independent).
    Returns O [B,Hq,R,dv] and LSE [B,Hq,R] (R = len(rows) or N)."""
    B, Hq, N, _ = q.shape
    G = Hq // k.shape[1]
    rows = np.arange(N) if rows is None else np.asarray(rows)
    O = np.zeros((B, Hq, len(rows), v.shape[-1]))
    LSE = np.zeros((B, Hq, len(rows)))
    internals = {}
    for b in range(B):
        for h in range(Hq):
            g = h // G
            Qh = _fq(q[b, h], -1, prec)
            Kh = _fq(k[b, g], -1, prec)
            Vc = _fq(v[b, g], 0, prec)
            s2 = (scale * (Qh[rows] @ Kh.T)) * LOG2E
            if causal:
                s2 = np.where(_future_mask(rows, N), -np.inf, s2)
            M = np.ceil(s2.max(axis=-1)) + max_shift
            p = np.exp2(s2 - M[:, None])
            l = p.sum(axis=-1)
            lse = (M + np.log2(l)) * LN2
            Ph = _fq(p, -1, prec)
            o = (Ph @ Vc) / l[:, None]
            if prec != "none":
                o = mxfp8.round_bf16(o)
                if not exact_stats:
                    lse = mxfp8.round_f32(lse)
            O[b, h] = o
            LSE[b, h] = lse
            if return_internals:
                internals[(b, h)] = dict(p=p, l=l, Ph=Ph, M=M)
    if return_internals:
        return O, LSE, internals
    return O, LSE


def _probabilities(q_row, k_row, lse, scale, causal, rows, cols):
    """P_ij = exp(S_ij - LSE_i) from the quantised Q, K and the saved LSE;
    future keys 0; not renormalised, not quantised (Appendix "Backward
    Correction and Gradient Computation")."""
    S = scale * (q_row[rows] @ k_row[cols].T)
    with np.errstate(over="ignore"):            # future keys may overflow before they are zeroed
        P = np.exp(S - np.asarray(lse, np.float64)[rows][:, None])
    if causal:
        P = np.where(np.asarray(cols)[None, :] > np.asarray(rows)[:, None], 0.0, P)
    return P


def emu_delta(q, k, v, dO, lse, scale, causal, prec="mxfp8", mode="matched", o=None,
              exact_stats=False, rows=None, dp_prec=None):
    """Row correction D [B,Hq,R].

    matched: D_i = sum_j P_ij dP^_ij with dP^ = dO^ V^^T from the row-blocked
             copies of dO and V (contraction over the value channels) -- Eq. 4.
    stale:   D_i = sum_k dO_ik O_ik from the BF16 dO and the saved BF16 O.
    consistent: the saved-output shortcut with dO replaced by the operand the backward matmuls
             consume, D_i = sum_k dO^_ik O_ik (paper Section 3.3, "consistent dO", Eq.
             delta_consistent_do_residual); dO^ is the row-blocked copy, the one dP^ uses.
    Stored FP32 unless ``exact_stats``."""
    B, Hq, N, _ = q.shape
    G = Hq // k.shape[1]
    rows = np.arange(N) if rows is None else np.asarray(rows)
    allc = np.arange(N)
    D = np.zeros((B, Hq, len(rows)))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            if mode == "stale":
                d = (mxfp8.round_bf16(dO[b, h])[rows] * np.asarray(o[b, h], np.float64)[rows]).sum(-1)
            elif mode == "consistent":
                d = (_fq(dO[b, h], -1, prec)[rows] * np.asarray(o[b, h], np.float64)[rows]).sum(-1)
            elif mode == "matched":
                P = _probabilities(_fq(q[b, h], -1, prec), _fq(k[b, g], -1, prec),
                                   lse[b, h], scale, causal, rows, allc)
                dP = _fq(dO[b, h], -1, dp_prec or prec)[rows] @ _fq(v[b, g], -1, dp_prec or prec).T
                d = (P * dP).sum(axis=-1)
            else:
                raise ValueError(mode)
            D[b, h] = d if exact_stats else mxfp8.round_f32(d)
    return D


def emu_backward(q, k, v, dO, lse, delta, scale, causal, prec="mxfp8", round_out=True,
                 return_internals=False, dp_prec=None):
    """Gradient pass given the saved LSE [B,Hq,N] and a row correction delta [B,Hq,N].

    Per head: S, P as in ``_probabilities``; dP^ = dO^r V^r^T (row-blocked
    copies); dS = P * (dP^ - delta) in full precision; then
      dV_g += P^i^T dO^c     P^i: P quantised in blocks of 32 query rows per key
      dK_g += scale dS^i^T Q^c   dS^i: dS quantised in blocks of 32 query rows
      dQ    = scale dS^j K^c     dS^j: dS quantised in blocks of 32 keys per row
    with ^c the copies of dO, Q, K blocked along tokens.  dK, dV are summed over
    the query heads of the group before rounding; all three are stored BF16.

    ``dp_prec`` overrides the operand precision of dP^ = dO V^T alone (the paper's protected-dP
    ablation, Appendix "Protected dP": dP from BF16 operands, the other products unchanged).

    Also returns the pre-cast row statistics sum_j dS_ij and sum_j |dS_ij|."""
    B, Hq, N, _ = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    allr = np.arange(N)
    dQ = np.zeros(q.shape)
    dK = np.zeros(k.shape)
    dV = np.zeros(v.shape)
    rowsum = np.zeros((B, Hq, N))
    rowabs = np.zeros((B, Hq, N))
    internals = {}
    for b in range(B):
        for h in range(Hq):
            g = h // G
            P = _probabilities(_fq(q[b, h], -1, prec), _fq(k[b, g], -1, prec),
                               lse[b, h], scale, causal, allr, allr)
            dP = _fq(dO[b, h], -1, dp_prec or prec) @ _fq(v[b, g], -1, dp_prec or prec).T
            dS = P * (dP - np.asarray(delta[b, h], np.float64)[:, None])
            rowsum[b, h] = dS.sum(axis=-1)
            rowabs[b, h] = np.abs(dS).sum(axis=-1)
            dV[b, g] += _fq(P, 0, prec).T @ _fq(dO[b, h], 0, prec)
            dK[b, g] += scale * (_fq(dS, 0, prec).T @ _fq(q[b, h], 0, prec))
            dQ[b, h] = scale * (_fq(dS, -1, prec) @ _fq(k[b, g], 0, prec))
            if return_internals:
                # dS_q / dS_k: the cast score gradients the dQ / dK matmuls consume (blocks of 32
                # keys per row / of 32 query rows per key)
                internals[(b, h)] = dict(P=P, dP=dP, dS=dS, dS_q=_fq(dS, -1, prec), dS_k=_fq(dS, 0, prec))
    if round_out and prec != "none":
        dQ, dK, dV = (mxfp8.round_bf16(x) for x in (dQ, dK, dV))
    out = (dQ, dK, dV, rowsum, rowabs)
    return out + (internals,) if return_internals else out


def emu_backward_rows(q, k, v, dO, lse, delta, scale, causal, b, h, rows, prec="mxfp8", dp_prec=None):
    """dQ rows and pre-cast row statistics of one head for some query rows
    (every query row of dQ is independent of the others).  ``lse`` and
    ``delta`` are that head's full [N] vectors."""
    N = q.shape[2]
    g = h // (q.shape[1] // k.shape[1])
    rows = np.asarray(rows)
    allc = np.arange(N)
    P = _probabilities(_fq(q[b, h], -1, prec), _fq(k[b, g], -1, prec), lse, scale, causal, rows, allc)
    dP = _fq(dO[b, h], -1, dp_prec or prec)[rows] @ _fq(v[b, g], -1, dp_prec or prec).T
    dS = P * (dP - np.asarray(delta, np.float64)[rows][:, None])
    dq = scale * (_fq(dS, -1, prec) @ _fq(k[b, g], 0, prec))
    return mxfp8.round_bf16(dq), dS.sum(-1), np.abs(dS).sum(-1)


def emu_backward_cols(q, k, v, dO, lse, delta, scale, causal, b, g, cols, prec="mxfp8", dp_prec=None):
    """dK and dV rows of one KV head for some keys (every key column of dS is
    independent of the others).  ``lse`` and ``delta`` are [Hq, N] for batch b."""
    N = q.shape[2]
    G = q.shape[1] // k.shape[1]
    cols = np.asarray(cols)
    allr = np.arange(N)
    dk = np.zeros((len(cols), k.shape[-1]))
    dv = np.zeros((len(cols), v.shape[-1]))
    for h in range(g * G, (g + 1) * G):
        P = _probabilities(_fq(q[b, h], -1, prec), _fq(k[b, g], -1, prec), lse[h], scale, causal, allr, cols)
        dP = _fq(dO[b, h], -1, dp_prec or prec) @ _fq(v[b, g], -1, dp_prec or prec)[cols].T
        dS = P * (dP - np.asarray(delta[h], np.float64)[:, None])
        dv += _fq(P, 0, prec).T @ _fq(dO[b, h], 0, prec)
        dk += scale * (_fq(dS, 0, prec).T @ _fq(q[b, h], 0, prec))
    return mxfp8.round_bf16(dk), mxfp8.round_bf16(dv)


def postcast_row_sums(q, k, v, dO, lse, delta, scale, causal, prec="mxfp8", rows=None, b=0, h=0):
    """Row sums of the CAST score gradient the dQ matmul consumes, dS'_ij (dS quantised in blocks of
    32 keys per row): sum_j dS'_ij and sum_j |dS'_ij| for one head (paper Appendix "dS Quantization
    Residuals", Eq. app_ds_quantization_residuals).  ``lse`` and ``delta`` are that head's [N] vectors."""
    N = q.shape[2]
    g = h // (q.shape[1] // k.shape[1])
    rows = np.arange(N) if rows is None else np.asarray(rows)
    allc = np.arange(N)
    P = _probabilities(_fq(q[b, h], -1, prec), _fq(k[b, g], -1, prec), lse, scale, causal, rows, allc)
    dP = _fq(dO[b, h], -1, prec)[rows] @ _fq(v[b, g], -1, prec).T
    dS = P * (dP - np.asarray(delta, np.float64)[rows][:, None])
    dSq = _fq(dS, -1, prec)
    return dSq.sum(axis=-1), np.abs(dSq).sum(axis=-1)


def postcast_residuals(rowsum_pre, rowabs_pre, rowsum_post, rowabs_post):
    """r_post = |sum dS'| / sum|dS|, r_post_own = |sum dS'| / sum|dS'| and the signed casting offset
    kappa = (sum dS' - sum dS) / sum|dS| (Eq. app_ds_quantization_residuals, app_ds_signed_increment);
    NaN where the denominator is zero."""
    with np.errstate(divide="ignore", invalid="ignore"):
        r_post = np.where(rowabs_pre > 0, np.abs(rowsum_post) / rowabs_pre, np.nan)
        r_own = np.where(rowabs_post > 0, np.abs(rowsum_post) / rowabs_post, np.nan)
        kappa = np.where(rowabs_pre > 0, (rowsum_post - rowsum_pre) / rowabs_pre, np.nan)
    return r_post, r_own, kappa


def key_common_mode(dK):
    """c_K = || sum_j dK_j ||_2 / ( sum_j ||dK_j||_2^2 )^(1/2) per (batch, KV head) for dK [B,Hkv,N,d]
    (Eq. app_ds_key_gradient_sum)."""
    dK = np.asarray(dK, np.float64)
    num = np.linalg.norm(dK.sum(axis=2), axis=-1)
    den = np.sqrt((dK ** 2).sum(axis=(2, 3)))
    return num / den


def residual_ratio(rowsum, rowabs):
    """r_i = |sum_j dS_ij| / sum_j |dS_ij| (pre-cast statistic of the paper's
    row-sum residual table); rows with a zero denominator give NaN."""
    with np.errstate(divide="ignore", invalid="ignore"):
        return np.where(rowabs > 0, np.abs(rowsum) / rowabs, np.nan)
