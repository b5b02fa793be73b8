"""Pins for the oracle's gated delta-rule recurrence (paper: Background, Eq. 1-2): closed forms of
the gates, pure decay, the overwrite property of the delta rule, the query scale and the impulse."""
import numpy as np

import oracle
from tests.golden.load import paper_constants

PC = paper_constants()


def _unit(rng, *shape):
    x = rng.standard_normal(shape)
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def test_gates_closed_forms():
    # softplus(0) = ln 2, A_log = 0 -> g = -ln 2 -> alpha = 1/2; sigmoid(0) = 1/2
    alpha, beta = oracle.gdn_gates(np.zeros((1, 1)), np.zeros((1, 1)), np.zeros(1), np.zeros(1))
    assert abs(alpha[0, 0] - 0.5) < 1e-15 and beta[0, 0] == 0.5
    # large a: softplus(a) -> a, alpha -> exp(-exp(A_log) a); very negative a: alpha -> 1
    alpha, _ = oracle.gdn_gates(np.array([[40.0, -40.0]]), np.zeros((1, 2)), np.log(np.array([0.01, 0.01])), np.zeros(2))
    assert abs(alpha[0, 0] - np.exp(-0.4)) < 1e-12 and 1.0 - alpha[0, 1] < 1e-15
    # dt_bias adds to a; sigmoid symmetry
    a1, b1 = oracle.gdn_gates(np.array([[0.3]]), np.array([[1.7]]), np.array([0.2]), np.array([0.5]))
    a2, b2 = oracle.gdn_gates(np.array([[0.8]]), np.array([[-1.7]]), np.array([0.2]), np.array([0.0]))
    assert a1[0, 0] == a2[0, 0] and abs(b1[0, 0] + b2[0, 0] - 1.0) < 1e-15
    assert np.all((a1 > 0) & (a1 < 1) & (b1 > 0) & (b1 < 1))


def test_pure_decay_and_pure_write():
    rng = np.random.default_rng(0)
    T, K = 6, 128
    k, q, v = _unit(rng, T, 1, K), _unit(rng, T, 1, K), rng.standard_normal((T, 1, K))
    A_log, dtb = np.zeros(1), np.zeros(1)
    # beta -> 0 after the first token: the state only decays, S_t = (prod alpha) S_0'
    b = np.full((T, 1), -800.0)
    b[0] = 800.0
    a = np.zeros((T, 1))
    S, _ = oracle.gdn_recurrence(q, k, v, a, b, A_log, dtb)
    assert np.allclose(S[0, 0], 0.5 * 0 + np.outer(k[0, 0], v[0, 0]), atol=1e-12)           # first write into an empty state
    for t in range(1, T):
        assert np.allclose(S[t, 0], 0.5 ** t * S[0, 0], rtol=1e-12, atol=1e-300)
    # alpha -> 1, beta -> 1: after writing (k, v) the state answers k with v exactly, and writing
    # the same pair again changes nothing (the delta rule corrects, it does not accumulate)
    a = np.full((T, 1), -800.0)
    b = np.full((T, 1), 800.0)
    k2 = np.repeat(k[:1], T, axis=0)
    v2 = np.repeat(v[:1], T, axis=0)
    S, o = oracle.gdn_recurrence(np.repeat(k[:1], T, axis=0), k2, v2, a, b, A_log, dtb)
    assert np.allclose(S[0, 0].T @ k[0, 0], v[0, 0], atol=1e-12)
    assert np.allclose(S[T - 1], S[0], atol=1e-12)
    # the query scale of Eq. 2: asking with q = k returns v / sqrt(K) (the appendix's 1 - 1/sqrt(128) = 91.2 % remark)
    assert np.allclose(o[0, 0], v[0, 0] / np.sqrt(K), atol=1e-12)
    assert abs((1 - 1 / np.sqrt(K)) - PC["missing_query_scale_output_difference"]) < 5e-4


def test_orthogonal_keys_store_independent_values_and_overwrite_key_by_key():
    K = 128
    eye = np.eye(K)
    T = 4
    k = eye[[0, 1, 0, 2]][:, None, :]                       # third token rewrites key 0
    v = np.arange(T * K, dtype=np.float64).reshape(T, 1, K)
    a = np.full((T, 1), -800.0)                             # no forgetting
    b = np.full((T, 1), 800.0)
    S, _ = oracle.gdn_recurrence(k, k, v, a, b, np.zeros(1), np.zeros(1))
    assert np.allclose(S[1, 0][0], v[0, 0]) and np.allclose(S[1, 0][1], v[1, 0])
    assert np.allclose(S[3, 0][0], v[2, 0])                 # overwritten, not summed
    assert np.allclose(S[3, 0][1], v[1, 0]) and np.allclose(S[3, 0][2], v[3, 0]) and np.all(S[3, 0][3:] == 0)


def test_shared_query_key_heads_and_impulse():
    rng = np.random.default_rng(1)
    T, Hk, Hv, K = 12, 2, 6, 128
    q, k = _unit(rng, T, Hk, K), _unit(rng, T, Hk, K)
    v = rng.standard_normal((T, Hv, K))
    a, b = rng.standard_normal((T, Hv)), rng.standard_normal((T, Hv))
    A_log, dtb = rng.standard_normal(Hv) * 0.3 - 2.0, rng.standard_normal(Hv) * 0.1
    S, o = oracle.gdn_recurrence(q, k, v, a, b, A_log, dtb)
    # value head 4 uses query/key head 4 // 3 = 1: recompute it alone
    S4, o4 = oracle.gdn_recurrence(q[:, 1:2], k[:, 1:2], v[:, 4:5], a[:, 4:5], b[:, 4:5], A_log[4:5], dtb[4:5])
    assert np.array_equal(S[:, 4], S4[:, 0]) and np.array_equal(o[:, 4], o4[:, 0])
    # a 1 % impulse at token 5 gives exactly 1 % state error there, nothing before, and a shrinking one after
    rs, _ = oracle.gdn_lockstep((q, k, v, a, b), (q, k, v, a, b), A_log, dtb, 1, impulse_step=5, impulse_rel=0.01)
    assert np.all(rs[:5] == 0) and np.allclose(rs[5], 0.01, rtol=1e-12)
    assert np.all(rs[6:] < 0.01) and np.all(np.diff(rs[5:], axis=0) < 0)
