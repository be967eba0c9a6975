"""Speculative-sampling arithmetic (Section 2; Algorithm 2 accept test and final draw).

Two layers live here, on purpose:

1. The *definition* in fp64 (``softmax64``, ``accept_probability``,
   ``residual_distribution``, ``acceptance_rate``): the formulas of Section 2
   written out.  Used for tolerance checks on probabilities and as the pin of
   layer 2.

2. The *decision arithmetic* (``exp_weights`` .. ``residual_sample``): the paper
   only says "sample r ~ U(0,1)" and "sample m ~ final_dist"; which token a
   given uniform maps to is fixed by this project, in the precision the CUDA
   kernels use, so that both sides take every integer decision identically and
   independently of summation order:

   * weights   E_k = min(floor(exp_spec(l_k - max l) * 2^32), 2^32 - 1), a 32-bit
               integer; exp_spec is a fixed sequence of IEEE fp32 operations (no
               fused multiply-add), written out in ``exp_weights``; tokens more
               than ~22.2 below the row maximum get weight 0;
   * totals    S = sum E_k (exact integer, < 2^64);
   * inverse CDF in ascending token id: tau = (U * S) >> 24, return the smallest k
               whose inclusive prefix sum exceeds tau (U is the 24-bit uniform);
   * fixed-point probabilities (units 2^-40): z = leading zeros of S as a 64-bit
               word, S'' = (S << z) >> 32, Rinv = floor((2^63 - 1) / S''),
               P_k = (E_k * Rinv) >> (55 - z);
   * accept iff ((U * P^q_x) >> 24) < P^p_x, i.e. u < p(x)/q(x) (the paper rejects
     when r > p/q; the two differ only on u == p/q);
   * residual weights r_k = max(0, P^p_k - P^q_k), drawn by the same inverse CDF;
     if they are all zero the draw falls back to the verifier's own row.

Layer 2 is pinned to layer 1 in tests/test_oracle_sampling.py (math.exp, exact
counts over the 2^24 uniforms, 1 - TV(p, q), the speculative-sampling lemma).
"""
import numpy as np

F32 = np.float32
SCALE_BITS = 32          # E_k = min(floor(w * 2^32), 2^32 - 1)
PROB_BITS = 40           # P_k in units of 2^-40
U_BITS = 24

# exp_spec constants, as fp32 bit patterns (part of the specification).
_LOG2E = np.array([0x3FB8AA3B], dtype=np.uint32).view(F32)[0]
_POLY = np.array([0x3F800000, 0x3F317215, 0x3E75FCDE, 0x3D635BA9, 0x3C1E7544, 0x3AADDD0A],
                 dtype=np.uint32).view(F32)   # 2^f on [-1/2, 1/2], ascending powers
_XMIN = F32(-32.0)


# ----------------------------------------------------------------------------- layer 1
def softmax64(logits):
    """Softmax at temperature 1 over the whole vocabulary, fp64."""
    l = np.asarray(logits, dtype=np.float64)
    w = np.exp(l - l.max())
    return w / w.sum()


def accept_probability(p, q, x):
    """min(1, p(x)/q(x)) (Section 2)."""
    return 1.0 if q[x] <= p[x] else float(p[x] / q[x])


def residual_distribution(p, q):
    """norm(max(0, p - q)) (Section 2, displayed formula); None if p == q."""
    r = np.maximum(0.0, np.asarray(p, np.float64) - np.asarray(q, np.float64))
    s = r.sum()
    return None if s == 0.0 else r / s


def acceptance_rate(p, q):
    """alpha_c = 1 - sum |p - q| / 2 (Section 2)."""
    return 1.0 - 0.5 * float(np.abs(np.asarray(p, np.float64) - np.asarray(q, np.float64)).sum())


def pairwise_acceptance(logits):
    """alpha[i][j] = mean over positions of the acceptance rate of drafter i under verifier j (Section 2's alpha
    between every pair of models, the input of the hierarchy search of Section 4.2).  logits: [models, rows, vocab]."""
    logits = np.asarray(logits, np.float64)
    L, R, _ = logits.shape
    probs = [[softmax64(logits[l, r]) for r in range(R)] for l in range(L)]
    alpha = np.ones((L, L))
    for i in range(L):
        for j in range(i + 1, L):
            alpha[i, j] = alpha[j, i] = sum(acceptance_rate(probs[i][r], probs[j][r]) for r in range(R)) / R
    return alpha


# ----------------------------------------------------------------------------- layer 2
def exp_weights(logits):
    """Integer softmax numerators E (uint64 array) of one row of stored logits.

    ``logits`` holds fp32-representable values (bf16 logits widen exactly).
    Every line below is one IEEE fp32 operation, round to nearest even.
    """
    l = np.asarray(logits, dtype=F32)
    m = l.max()
    x = l - m                                   # fp32 subtract
    x = np.maximum(x, _XMIN)                    # clamp so that 2^j stays a normal number
    t = x * _LOG2E                              # fp32 multiply
    j = np.rint(t)                              # round half to even, exact
    f = t - j                                   # exact, in [-1/2, 1/2]
    p = np.full_like(f, _POLY[5])
    for c in (_POLY[4], _POLY[3], _POLY[2], _POLY[1], _POLY[0]):
        p = p * f                               # fp32 multiply
        p = p + c                               # fp32 add
    w = np.ldexp(p, (j.astype(np.int32) + SCALE_BITS))   # exact power-of-two scaling
    e = np.minimum(np.floor(w).astype(np.float64), 4294967295.0)
    return e.astype(np.uint64)


def fixed_probs(E):
    """Fixed-point probabilities P (uint64 array, units 2^-40) and the total S."""
    S = int(E.sum(dtype=np.uint64))
    z = 64 - S.bit_length()                      # S >= 2^32 - 1, so 0 <= z <= 32
    s_top = ((S << z) & 0xFFFFFFFFFFFFFFFF) >> 32  # in [2^31, 2^32)
    rinv = ((1 << 63) - 1) // s_top              # < 2^32, and E < 2^32: the product fits 64 bits
    P = (E * np.uint64(rinv)) >> np.uint64(55 - z)
    return P, S


def inverse_cdf(weights, total, U):
    """Smallest k with sum_{k' <= k} weights[k'] > (U * total) >> 24."""
    tau = (int(U) * int(total)) >> U_BITS
    c = 0
    for k, w in enumerate(weights.tolist()):
        c += w
        if c > tau:
            return k
    raise AssertionError("unreachable: U < 2^24 implies tau < total")


def inverse_cdf_fast(weights, total, U):
    """Same result as ``inverse_cdf`` via an exact integer cumulative sum."""
    tau = (int(U) * int(total)) >> U_BITS
    c = np.cumsum(weights.astype(np.uint64), dtype=np.uint64)
    return int(np.searchsorted(c, np.uint64(tau), side="right"))


def categorical(logits, U):
    """x ~ softmax(logits) by the inverse CDF over the integer weights."""
    E = exp_weights(logits)
    return inverse_cdf_fast(E, int(E.sum(dtype=np.uint64)), U)


def accept(Pp_x, Pq_x, U):
    """Accept iff u < p(x)/q(x), in fixed point."""
    return ((int(U) * int(Pq_x)) >> U_BITS) < int(Pp_x)


def residual_sample(p_logits, q_logits, U):
    """m ~ norm(max(0, p - q)); falls back to m ~ p when the residual is all zero."""
    Ep = exp_weights(p_logits)
    Eq = exp_weights(q_logits)
    Pp, Sp = fixed_probs(Ep)
    Pq, _ = fixed_probs(Eq)
    r = np.where(Pp > Pq, Pp - Pq, np.uint64(0))
    total = int(r.sum(dtype=np.uint64))
    if total == 0:
        return inverse_cdf_fast(Ep, Sp, U)
    return inverse_cdf_fast(r, total, U)
