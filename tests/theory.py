"""Closed forms and bounds from the paper, written independently of oracle/ and of the CUDA path.

Used only by the tests, as the yardstick the oracle (and through it the kernels) is held to.
"""
import numpy as np
from scipy import integrate


def softmax(x):
    x = np.asarray(x, dtype=np.float64)
    e = np.exp(x - x.max())
    return e / e.sum()


def lml_bound(p, q, K):
    """Theorem 1, unconditional list matching lemma:
    sum_j K / sum_i [max(q_i/q_j, p_i/p_j) + (K-1) q_i/q_j]   (terms with p_j = 0 or q_j = 0 drop)."""
    p = np.asarray(p, float)
    q = np.asarray(q, float)
    tot = 0.0
    for j in range(len(p)):
        if p[j] <= 0 or q[j] <= 0:
            continue
        den = np.sum(np.maximum(q / q[j], p / p[j]) + (K - 1) * q / q[j])
        tot += K / den
    return tot


def lml_conditional_relaxed(p, q, K):
    """Relaxed form below Theorem 1's proof: sum_j q_j (1 + q_j/(K p_j))^-1."""
    p = np.asarray(p, float)
    q = np.asarray(q, float)
    m = (p > 0) & (q > 0)
    return float(np.sum(q[m] / (1.0 + q[m] / (K * p[m]))))


def joint_flat_first(p, q, K, j):
    """Proof of Theorem 1: Pr[Y~ = j, X^(1) = j] = 1 / sum_i [max(q_i/q_j, p_i/p_j) + (K-1) q_i/q_j],
    where Y~ = j means that stream 1 achieved the target minimum at token j."""
    p = np.asarray(p, float)
    q = np.asarray(q, float)
    return 1.0 / np.sum(np.maximum(q / q[j], p / p[j]) + (K - 1) * q / q[j])


def k1_acceptance(p, q):
    """Remark after Theorem 1 (K = 1 is tight): Pr[Y = X] = sum_j 1 / sum_i max(q_i/q_j, p_i/p_j)."""
    return lml_bound(p, q, 1)


def exact_acceptance(p, q, K):
    """Exact Pr[Y in {X^(1..K)}] for full-support p, q, by quadrature.

    Derivation (same flattening as the proof of Theorem 1, then the memoryless property):
    condition on the winning pair (token j, stream 1) and on the winning value t = S_j^(1)/q_j, whose
    joint density is q_j exp(-K t); every other S_i^(k) is then t q_i plus a fresh Exp(1).
      - stream 1 proposes j  iff  every fresh e_i >= t (p_i q_j / p_j - q_i):  prob exp(-t D_j),
        D_j = sum_i max(0, p_i q_j/p_j - q_i);
      - stream k >= 2 proposes j with prob a_j(t) = int_0^inf e^-r prod_{i != j}
        exp(-max(0, t (p_i q_j/p_j - q_i) + r p_i/p_j)) dr   (r = the fresh part of S_j^(k)).
    Streams are independent given (j, t), and the K choices of the winning stream are symmetric:
      Pr[acc] = K sum_j q_j int_0^inf e^{-K t} [1 - (1 - e^{-t D_j}) (1 - a_j(t))^{K-1}] dt.
    Dropping the a_j factor gives Theorem 1's bound; K = 1 gives the K = 1 closed form.
    """
    p = np.asarray(p, float)
    q = np.asarray(q, float)
    n = len(p)
    total = 0.0
    for j in range(n):
        c = p * q[j] / p[j] - q  # slope in t
        d = p / p[j]  # slope in r
        Dj = np.sum(np.maximum(0.0, c))
        others = [i for i in range(n) if i != j]

        def a_j(t):
            if K == 1:
                return 0.0

            def inner(r):
                return np.exp(-r - sum(max(0.0, t * c[i] + r * d[i]) for i in others))

            val, _ = integrate.quad(inner, 0.0, np.inf, epsabs=1e-11, epsrel=1e-10)
            return val

        def outer(t):
            miss = (1.0 - np.exp(-t * Dj)) * (1.0 - a_j(t)) ** (K - 1)
            return np.exp(-K * t) * (1.0 - miss)

        val, _ = integrate.quad(outer, 0.0, np.inf, epsabs=1e-10, epsrel=1e-9)
        total += K * q[j] * val
    return total


def lml_bound_active(p, q, K, J):
    """Appendix B: with J of the K coupled drafts still active, the probability that the target
    token (min over ALL K streams) matches an active draft is at least
    sum_j J / sum_i [max(q_i/q_j, p_i/p_j) + (K-1) q_i/q_j]."""
    return lml_bound(p, q, K) * J / K


def exact_acceptance_active(p, q, K, J):
    """Exact Pr[Y in {X^(1..J)}] when Y is the target race over all K streams and only J of the
    K proposals count (Appendix B's setting), by the same conditioning as exact_acceptance():
    given the winning pair (token j, value t), the winning stream is one of the J active ones
    with probability J/K -- then the match fails only if that stream misses j (1 - e^{-t D_j})
    and so do the other J-1 active ones -- or one of the K-J inactive ones, where all J active
    streams must miss:
      Pr = sum_j q_j int_0^inf e^{-K t} [ J (1 - (1 - e^{-t D_j}) (1 - a_j)^{J-1})
                                          + (K - J) (1 - (1 - a_j)^J) ] dt."""
    p = np.asarray(p, float)
    q = np.asarray(q, float)
    n = len(p)
    total = 0.0
    for j in range(n):
        c = p * q[j] / p[j] - q
        d = p / p[j]
        Dj = np.sum(np.maximum(0.0, c))
        others = [i for i in range(n) if i != j]

        def a_j(t):
            def inner(r):
                return np.exp(-r - sum(max(0.0, t * c[i] + r * d[i]) for i in others))

            val, _ = integrate.quad(inner, 0.0, np.inf, epsabs=1e-11, epsrel=1e-10)
            return val

        def outer(t):
            a = a_j(t)
            win_active = 1.0 - (1.0 - np.exp(-t * Dj)) * (1.0 - a) ** (J - 1)
            win_inactive = 1.0 - (1.0 - a) ** J
            return np.exp(-K * t) * (J * win_active + (K - J) * win_inactive)

        val, _ = integrate.quad(outer, 0.0, np.inf, epsabs=1e-10, epsrel=1e-9)
        total += q[j] * val
    return total
