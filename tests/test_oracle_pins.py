"""Pins for the fp64 CPU oracle: closed forms, invariants, special cases that reduce to
library routines, brute force on tiny inputs, and independent restatements.  None of
these re-types the oracle's own loop; a dropped term, a wrong sign or index, a
transposed state or a swapped decay/update order fails at least one of them."""
import numpy as np
import pytest

import oracle
from oracle import reformulations as R
from gdn_inputs import bf16_bits_to_f32, f32_to_bf16_bits, make_cu_seqlens, make_state, make_tokens, config
from helpers import head_view, rel_fro, round_bf16


def run_single(q, k, v, g, beta, S0=None, cu=None):
    """Call the C oracle on one head given fp64 arrays that are exactly representable
    (q,k,v in bf16; g,beta,S0 in fp32)."""
    T, dk = q.shape
    dv = v.shape[1]
    qb, kb, vb = (f32_to_bf16_bits(x.astype(np.float32)).reshape(T, 1, -1) for x in (q, k, v))
    for bits, x in ((qb, q), (kb, k), (vb, v)):
        assert np.array_equal(bf16_bits_to_f32(bits).reshape(x.shape).astype(np.float64), x), "input not bf16-exact"
    g32, b32 = g.astype(np.float32).reshape(T, 1), beta.astype(np.float32).reshape(T, 1)
    assert np.array_equal(g32.astype(np.float64).ravel(), g) and np.array_equal(b32.astype(np.float64).ravel(), beta)
    if cu is None:
        cu = make_cu_seqlens([T])
    N = len(cu) - 1
    init = None if S0 is None else np.asarray(S0, dtype=np.float32).reshape(N, 1, dv, dk)
    out, fin = oracle.prefill(qb, kb, vb, g32, b32, cu, init, threads=2)
    return out[:, 0, :], fin[:, 0]


def rand_head(T, dk, dv, seed, S0=True, gate_mean=1.0):
    rng = np.random.default_rng(seed)
    _, q = round_bf16(rng.standard_normal((T, dk)) / np.sqrt(dk))
    kraw = rng.standard_normal((T, dk))
    _, k = round_bf16(kraw / np.linalg.norm(kraw, axis=1, keepdims=True))
    _, v = round_bf16(rng.standard_normal((T, dv)))
    x = rng.standard_normal(T) + gate_mean
    g = (-np.log1p(np.exp(-x))).astype(np.float32).astype(np.float64)
    beta = (1 / (1 + np.exp(-rng.standard_normal(T)))).astype(np.float32).astype(np.float64)
    S = (0.3 * rng.standard_normal((dv, dk))).astype(np.float32).astype(np.float64) if S0 else np.zeros((dv, dk))
    return q, k, v, g, beta, S


# ---- I1: one token from the zero state: S = beta v k^T, o = beta v (k.q); alpha drops out
def test_one_token_closed_form():
    q, k, v, g, beta, _ = rand_head(1, 16, 8, 1, S0=False)
    out, fin = run_single(q, k, v, g, beta)
    np.testing.assert_allclose(fin[0], beta[0] * np.outer(v[0], k[0]), rtol=0, atol=1e-15)
    np.testing.assert_allclose(out[0], beta[0] * v[0] * (k[0] @ q[0]), rtol=0, atol=1e-15)
    # orientation: rows follow v, columns follow k (dk != dv here, so a transpose cannot pass)
    assert fin[0].shape == (8, 16)


# ---- I2: beta = 0 is pure decay: S_t = exp(sum g) S0, o_t = exp(gamma_t) S0 q_t
def test_beta_zero_pure_decay():
    q, k, v, g, beta, S0 = rand_head(9, 8, 5, 2)
    beta[:] = 0.0
    out, fin = run_single(q, k, v, g, beta, S0)
    gam = np.cumsum(g)
    np.testing.assert_allclose(fin[0], np.exp(gam[-1]) * S0, rtol=1e-14)
    np.testing.assert_allclose(out, np.exp(gam)[:, None] * (q @ S0.T), rtol=1e-13, atol=1e-16)


# ---- I3: g = 0, beta = 1, one-hot keys: associative memory, exact retrieval and overwrite
def test_onehot_keys_associative_recall():
    dk, dv, T = 8, 5, 6
    rng = np.random.default_rng(3)
    slots = [2, 5, 0, 7, 5, 3]  # slot 5 is written twice: the second write overwrites
    k = np.zeros((T, dk))
    k[np.arange(T), slots] = 1.0
    _, v = round_bf16(rng.standard_normal((T, dv)))
    q = k.copy()
    g = np.zeros(T)
    beta = np.ones(T)
    S0 = (0.5 * rng.standard_normal((dv, dk))).astype(np.float32).astype(np.float64)
    out, fin = run_single(q, k, v, g, beta, S0)
    # S_t k_t = v_t exactly right after the write
    np.testing.assert_array_equal(out, v)
    expect = S0.copy()
    for t, s in enumerate(slots):
        expect[:, s] = v[t]
    np.testing.assert_array_equal(fin[0], expect)
    # querying an earlier key later retrieves its (latest) value
    q2 = np.zeros((T, dk))
    q2[:, 2] = 1.0
    out2, _ = run_single(q2, k, v, g, beta, S0)
    np.testing.assert_array_equal(out2, np.repeat(v[0:1], T, axis=0))


# ---- I4: per-step identity S_t k_t = alpha (1 - beta |k|^2) S_{t-1} k_t + beta |k|^2 v_t
def test_one_step_key_identity():
    q, k, v, g, beta, S0 = rand_head(12, 16, 8, 4)
    S_prev = S0
    for t in range(12):
        # use q = k so that the oracle's output *is* S_t k_t
        out, fin = run_single(k[t:t + 1], k[t:t + 1], v[t:t + 1], g[t:t + 1], beta[t:t + 1], S_prev)
        n2 = k[t] @ k[t]
        expect = np.exp(g[t]) * (1 - beta[t] * n2) * (S_prev @ k[t]) + beta[t] * n2 * v[t]
        np.testing.assert_allclose(out[0], expect, rtol=1e-13, atol=1e-15)
        S_prev = fin[0].astype(np.float32).astype(np.float64)  # hand over as the fp32 state a caller would hold


# ---- I5: pairwise-orthogonal keys -> gated linear attention through three library matmuls
def test_orthogonal_keys_reduce_to_linear_attention():
    dk, dv, T = 16, 8, 11
    rng = np.random.default_rng(5)
    perm = rng.permutation(dk)[:T]
    k = np.zeros((T, dk))
    k[np.arange(T), perm] = 1.0
    q, _, v, g, beta, S0 = rand_head(T, dk, dv, 6)
    out, fin = run_single(q, k, v, g, beta, S0)
    o2, s2 = R.orthogonal_keys_closed_form(q, k, v, g, beta, S0)
    np.testing.assert_allclose(out, o2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(fin[0], s2, rtol=1e-12, atol=1e-14)


# ---- I6: split / hand-off / packing invariance, and prefill == repeated decode
def test_split_and_packing_invariance():
    tok = make_tokens(37, 2, 4, dk=8, dv=6, seed=11, gate_mean=1.0)
    init = make_state(1, 4, 8, 6, seed=11, sd=0.3)
    full_o, full_s = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, make_cu_seqlens([37]), init)
    T1 = 13
    o1, s1 = oracle.prefill(tok.q[:T1], tok.k[:T1], tok.v[:T1], tok.g[:T1], tok.beta[:T1], make_cu_seqlens([T1]), init)
    # the hand-over state stays fp64 here by re-running from the fp32-rounded state on both sides
    s1_32 = s1.astype(np.float32)
    o2, s2 = oracle.prefill(tok.q[T1:], tok.k[T1:], tok.v[T1:], tok.g[T1:], tok.beta[T1:], make_cu_seqlens([37 - T1]), s1_32)
    np.testing.assert_allclose(o1, full_o[:T1], rtol=0, atol=0)
    assert rel_fro(o2, full_o[T1:]) < 1e-6 and rel_fro(s2, full_s) < 1e-6  # only the fp32 hand-over rounds
    # packing: two sequences in one call == two calls
    cu = make_cu_seqlens([T1, 37 - T1])
    init2 = np.concatenate([init, s1_32], axis=0)
    op, sp = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cu, init2)
    np.testing.assert_array_equal(op[:T1], o1)
    np.testing.assert_array_equal(op[T1:], o2)
    np.testing.assert_array_equal(sp[0], s1[0])
    np.testing.assert_array_equal(sp[1], s2[0])


def test_prefill_equals_repeated_decode():
    tok = make_tokens(5, 1, 2, dk=8, dv=4, seed=12)
    init = make_state(1, 2, 8, 4, seed=12, sd=0.3)
    full_o, full_s = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, make_cu_seqlens([5]), init)
    S = init.astype(np.float64)
    for t in range(5):
        # decode takes an fp32 state: keep the comparison exact by checking one step at a time
        S32 = S.astype(np.float32)
        o, S = oracle.decode(tok.q[t:t + 1], tok.k[t:t + 1], tok.v[t:t + 1], tok.g[t:t + 1], tok.beta[t:t + 1], S32)
        o_ref, S_ref = oracle.prefill(tok.q[t:t + 1], tok.k[t:t + 1], tok.v[t:t + 1], tok.g[t:t + 1], tok.beta[t:t + 1],
                                      make_cu_seqlens([1]), S32)
        np.testing.assert_array_equal(o, o_ref)
        np.testing.assert_array_equal(S, S_ref)
    assert rel_fro(S, full_s) < 1e-6


def test_decode_batch_items_are_independent_sequences():
    tok = make_tokens(6, 2, 4, dk=8, dv=4, seed=13)
    st = make_state(6, 4, 8, 4, seed=13, sd=0.3)
    o, s = oracle.decode(tok.q, tok.k, tok.v, tok.g, tok.beta, st)
    o2, s2 = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, make_cu_seqlens([1] * 6), st)
    np.testing.assert_array_equal(o, o2)
    np.testing.assert_array_equal(s, s2)


# ---- I7: linearity in (S0, V) and in q
def test_linearity():
    q, k, v, g, beta, S0 = rand_head(10, 8, 6, 20)
    _, _, v2, _, _, S02 = rand_head(10, 8, 6, 21)
    oa, sa = run_single(q, k, v, g, beta, S0)
    ob, sb = run_single(q, k, v2, g, beta, S02)
    # scaling by 0.5 / 2.0 keeps every input exactly representable
    oc, sc = run_single(q, k, 0.5 * v, g, beta, 0.5 * S0)
    np.testing.assert_allclose(oc, 0.5 * oa, rtol=1e-13, atol=1e-16)
    np.testing.assert_allclose(sc[0], 0.5 * sa[0], rtol=1e-13, atol=1e-16)
    # superposition with the zero-input response: (S0+S02, v+v2) is not bf16-exact in general,
    # so superpose in the state only (fp32-exact sums of fp32 halves)
    S_sum = (0.5 * S0 + 0.5 * S02)
    if np.array_equal(S_sum.astype(np.float32).astype(np.float64), S_sum):
        od, sd = run_single(q, k, np.zeros_like(v), g, beta, S_sum)
        oe, se = run_single(q, k, np.zeros_like(v), g, beta, S0)
        of, sf = run_single(q, k, np.zeros_like(v), g, beta, S02)
        np.testing.assert_allclose(od, 0.5 * oe + 0.5 * of, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(sd[0], 0.5 * se[0] + 0.5 * sf[0], rtol=1e-12, atol=1e-15)
    og, _ = run_single(2.0 * q, k, v, g, beta, S0)
    np.testing.assert_allclose(og, 2.0 * oa, rtol=1e-13, atol=1e-16)
    assert ob.shape == oa.shape and sb.shape == sa.shape


# ---- I8: V-row independence: row r of S and column r of o depend only on v[:,r] and S0[r,:]
def test_v_row_independence():
    q, k, v, g, beta, S0 = rand_head(9, 8, 6, 30)
    oa, sa = run_single(q, k, v, g, beta, S0)
    v2, S2 = v.copy(), S0.copy()
    v2[:, 3] = -v2[:, 3]
    S2[3, :] = 0.25
    ob, sb = run_single(q, k, v2, g, beta, S2)
    keep = [0, 1, 2, 4, 5]
    np.testing.assert_array_equal(oa[:, keep], ob[:, keep])
    np.testing.assert_array_equal(sa[0][keep], sb[0][keep])
    assert not np.allclose(oa[:, 3], ob[:, 3])
    # and a single row run alone reproduces that row
    oc, sc = run_single(q, k, v[:, 3:4], g, beta, S0[3:4])
    np.testing.assert_array_equal(oc[:, 0], oa[:, 3])
    np.testing.assert_array_equal(sc[0][0], sa[0][3])


# ---- I9: brute force on tiny inputs + the paper's K x V form coded separately
@pytest.mark.parametrize("T,dk,dv,seed", [(1, 2, 3, 40), (5, 4, 3, 41), (8, 3, 4, 42)])
def test_bruteforce_and_paper_form(T, dk, dv, seed):
    q, k, v, g, beta, S0 = rand_head(T, dk, dv, seed)
    out, fin = run_single(q, k, v, g, beta, S0)
    o1, s1 = R.explicit_product(q, k, v, g, beta, S0)
    o2, s2 = R.paper_form(q, k, v, g, beta, S0)
    np.testing.assert_allclose(out, o1, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(fin[0], s1, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(out, o2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(fin[0], s2, rtol=1e-12, atol=1e-14)


def test_paper_form_on_longer_random_run():
    q, k, v, g, beta, S0 = rand_head(150, 32, 16, 43)
    out, fin = run_single(q, k, v, g, beta, S0)
    o2, s2 = R.paper_form(q, k, v, g, beta, S0)
    assert rel_fro(out, o2) < 1e-13 and rel_fro(fin[0], s2) < 1e-13


# ---- I10: chunked WY/UT form agrees with the sequential definition, for any chunk size
@pytest.mark.parametrize("T", [1, 63, 64, 65, 130])
@pytest.mark.parametrize("C", [4, 16, 64])
def test_chunked_reformulation(T, C):
    q, k, v, g, beta, S0 = rand_head(T, 16, 8, 50 + T)
    out, fin = run_single(q, k, v, g, beta, S0)
    o2, s2 = R.chunked(q, k, v, g, beta, S0, C=C)
    assert rel_fro(out, o2) < 1e-12 and rel_fro(fin[0], s2) < 1e-12


def test_chunked_reformulation_on_tiny_config():
    cfg = config("prefill_tiny")
    tok = cfg["tokens"]
    out, fin = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cfg["cu_seqlens"], None)
    q, k, v, g, b = head_view(tok, 0, 64, 0)
    o2, s2 = R.chunked(q, k, v, g, b, np.zeros((128, 128)), C=64)
    assert rel_fro(out[:, 0], o2) < 1e-12 and rel_fro(fin[0, 0], s2) < 1e-12
    o3, s3 = R.chunked(q, k, v, g, b, np.zeros((128, 128)), C=16)
    assert rel_fro(o3, o2) < 1e-12 and rel_fro(s3, s2) < 1e-12


# ---- I11: contraction bound |S_t|_F <= |S_{t-1}|_F + beta |v| |k| for |k|<=1, beta in [0,1], g<=0
def test_contraction_bound():
    q, k, v, g, beta, S0 = rand_head(40, 16, 8, 60)
    k = k * 0.5  # still bf16-exact, norm < 1
    S = S0
    for t in range(40):
        _, fin = run_single(q[t:t + 1], k[t:t + 1], v[t:t + 1], g[t:t + 1], beta[t:t + 1], S)
        bound = np.linalg.norm(S) + beta[t] * np.linalg.norm(v[t]) * np.linalg.norm(k[t])
        assert np.linalg.norm(fin[0]) <= bound * (1 + 1e-12)
        S = fin[0].astype(np.float32).astype(np.float64)


# ---- head mapping (grouped value heads): value heads 2j, 2j+1 read q/k head j
def test_grouped_head_mapping_is_blocked():
    tok = make_tokens(7, 2, 4, dk=8, dv=4, seed=70)
    out, fin = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, make_cu_seqlens([7]), None)
    for h in range(4):
        q, k, v, g, b = head_view(tok, 0, 7, h)  # head_view maps h -> h // 2
        o2, s2 = R.paper_form(q, k, v, g, b, np.zeros((4, 8)))
        assert rel_fro(out[:, h], o2) < 1e-13 and rel_fro(fin[0, h], s2) < 1e-13


# ---- zero-length sequences and empty batches
def test_zero_length_sequence_and_empty_batch():
    tok = make_tokens(5, 1, 1, dk=4, dv=4, seed=80)
    init = make_state(3, 1, 4, 4, seed=80, sd=0.3)
    cu = make_cu_seqlens([2, 0, 3])
    out, fin = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cu, init)
    np.testing.assert_array_equal(fin[1], init[1].astype(np.float64))
    o_a, f_a = oracle.prefill(tok.q[:2], tok.k[:2], tok.v[:2], tok.g[:2], tok.beta[:2], make_cu_seqlens([2]), init[0:1])
    np.testing.assert_array_equal(out[:2], o_a)
    np.testing.assert_array_equal(fin[0], f_a[0])
    e = make_tokens(0, 1, 1, dk=4, dv=4, seed=81)
    o_e, f_e = oracle.prefill(e.q, e.k, e.v, e.g, e.beta, make_cu_seqlens([]), None)
    assert o_e.shape == (0, 1, 4) and f_e.shape == (0, 1, 4, 4)


def test_thread_count_does_not_change_results():
    tok = make_tokens(20, 2, 4, dk=8, dv=8, seed=90)
    cu = make_cu_seqlens([7, 13])
    init = make_state(2, 4, 8, 8, seed=90)
    a = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cu, init, threads=1)
    b = oracle.prefill(tok.q, tok.k, tok.v, tok.g, tok.beta, cu, init, threads=5)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


# ---- raw-gate form (Section 3.2): g = exp(-exp(A_log) softplus(a + dt_bias)), beta = sigmoid(b)
def test_gated_oracle_closed_forms_and_agreement_with_the_ungated_form():
    from gdn_inputs import make_raw_gates
    tok = make_tokens(12, 1, 2, dk=8, dv=4, seed=100)
    a, b, A_log, dt_bias = make_raw_gates(12, 2, seed=100)
    init = make_state(1, 2, 8, 4, seed=100, sd=0.3)
    cu = make_cu_seqlens([12])
    # closed forms: a + dt_bias = 0 -> softplus = ln 2, so alpha = exp(-A ln 2) = 2^-A; b = 0 -> beta = 1/2
    a0 = np.zeros_like(a) - dt_bias[None, :]
    A_two = np.log(np.array([1.0, 3.0], dtype=np.float32)).astype(np.float32)
    o, s = oracle.prefill_gated(tok.q, tok.k, tok.v, a0, np.zeros_like(b), A_two, dt_bias, cu, init)
    alpha = np.broadcast_to(np.array([0.5, 0.125]), (12, 2))
    # dt_bias is fp32 and a0 = -dt_bias exactly, so a + dt_bias is exactly 0
    o2, s2 = oracle.prefill(tok.q, tok.k, tok.v, np.log(alpha).astype(np.float32), np.full((12, 2), 0.5, np.float32), cu, init)
    assert rel_fro(o, o2) < 1e-7 and rel_fro(s, s2) < 1e-7   # only log(0.5) rounded to fp32 differs
    # general inputs: gates computed here in fp64 with library functions, rounded to fp32, fed to the ungated form
    x = a.astype(np.float64) + dt_bias.astype(np.float64)[None, :]
    g64 = -np.exp(A_log.astype(np.float64))[None, :] * np.logaddexp(0.0, x)
    beta64 = 1.0 / (1.0 + np.exp(-b.astype(np.float64)))
    o3, s3 = oracle.prefill_gated(tok.q, tok.k, tok.v, a, b, A_log, dt_bias, cu, init)
    o4, s4 = oracle.prefill(tok.q, tok.k, tok.v, g64.astype(np.float32), beta64.astype(np.float32), cu, init)
    assert rel_fro(o3, o4) < 1e-6 and rel_fro(s3, s4) < 1e-6
    # extremes: very negative a + dt_bias -> no decay; very positive b -> beta -> 1
    o5, s5 = oracle.prefill_gated(tok.q, tok.k, tok.v, np.full_like(a, -80.0), np.full_like(b, 80.0), A_log, dt_bias, cu, init)
    o6, s6 = oracle.prefill(tok.q, tok.k, tok.v, np.zeros_like(a), np.ones_like(b), cu, init)
    assert rel_fro(o5, o6) < 1e-12 and rel_fro(s5, s6) < 1e-12
    # decode form agrees with a one-token prefill
    st = make_state(12, 2, 8, 4, seed=101, sd=0.3)
    od, sd = oracle.decode_gated(tok.q, tok.k, tok.v, a, b, A_log, dt_bias, st)
    op, sp = oracle.prefill_gated(tok.q, tok.k, tok.v, a, b, A_log, dt_bias, make_cu_seqlens([1] * 12), st)
    np.testing.assert_array_equal(od, op)
    np.testing.assert_array_equal(sd, sp)


# ---- affine in the state (the identity behind sequence-parallel prefill): with M_t the product of the
#      per-token transitions and H_t the zero-state response,  S_t = S_in M_t + H_t,  o_t = H_t q_t + S_in (M_t q_t).
#      M_t q_t and M_T come from running the oracle itself on the identity (dk x dk "state", v = 0).
def test_state_enters_affinely_through_the_transition_product():
    T, dk, dv = 23, 8, 5
    q, k, v, g, beta, S_in = rand_head(T, dk, dv, 41)
    o_full, s_full = run_single(q, k, v, g, beta, S_in)
    o_zero, s_zero = run_single(q, k, v, g, beta, None)                           # H_t q_t, H_T
    o_id, s_id = run_single(q, k, np.zeros((T, dk)), g, beta, np.eye(dk))         # M_t q_t, M_T (a dk x dk run)
    np.testing.assert_allclose(o_full, o_zero + o_id @ S_in.T, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(s_full[0], S_in @ s_id[0] + s_zero[0], rtol=1e-12, atol=1e-14)
    # and the transition product itself, written out: M_T = prod_t alpha_t (I - beta_t k_t k_t^T)
    M = np.eye(dk)
    for t in range(T):
        M = np.exp(g[t]) * (M @ (np.eye(dk) - beta[t] * np.outer(k[t], k[t])))
    np.testing.assert_allclose(s_id[0], M, rtol=1e-12, atol=1e-14)
    # two pieces joined: state after piece 1 enters piece 2
    T1 = 9
    _, s1 = run_single(q[:T1], k[:T1], v[:T1], g[:T1], beta[:T1], S_in)
    o2_zero, s2_zero = run_single(q[T1:], k[T1:], v[T1:], g[T1:], beta[T1:], None)
    o2_id, s2_id = run_single(q[T1:], k[T1:], np.zeros((T - T1, dk)), g[T1:], beta[T1:], np.eye(dk))
    np.testing.assert_allclose(o_full[T1:], o2_zero + o2_id @ s1[0].T, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(s_full[0], s1[0] @ s2_id[0] + s2_zero[0], rtol=1e-12, atol=1e-14)


# ---- fused front end: q/k L2 normalisation (x / sqrt(sum x^2 + 1e-6)) and a scale on q
def test_fused_front_end_scale_normalisation_and_recall():
    tok = make_tokens(40, 2, 4, dk=16, dv=6, seed=200)
    # make the norms far from 1 and different per token, exactly in bf16 (powers of two per token)
    rng = np.random.default_rng(200)
    pw_k = (2.0 ** rng.integers(-2, 4, size=(40, 2, 1))).astype(np.float32)
    pw_q = (2.0 ** rng.integers(-3, 3, size=(40, 2, 1))).astype(np.float32)
    kb = f32_to_bf16_bits(bf16_bits_to_f32(tok.k) * pw_k)
    qb = f32_to_bf16_bits(bf16_bits_to_f32(tok.q) * pw_q)
    init = make_state(2, 4, 16, 6, seed=200, sd=0.3)
    cu = make_cu_seqlens([29, 11])
    # (1) switched off it is the plain definition, bit for bit
    o0, s0 = oracle.prefill(qb, kb, tok.v, tok.g, tok.beta, cu, init)
    o1, s1 = oracle.prefill_fused(qb, kb, tok.v, tok.g, tok.beta, None, None, cu, init, scale=1.0, qk_l2norm=False)
    np.testing.assert_array_equal(o0, o1)
    np.testing.assert_array_equal(s0, s1)
    # (2) scale multiplies the outputs and leaves the states alone (o = S q is linear in q; S does not see q)
    o2, s2 = oracle.prefill_fused(qb, kb, tok.v, tok.g, tok.beta, None, None, cu, init, scale=0.375, qk_l2norm=False)
    np.testing.assert_allclose(o2, 0.375 * o0, rtol=1e-13, atol=1e-300)
    np.testing.assert_array_equal(s2, s0)
    # (3) normalisation: the separately coded forms, fed inputs normalised here with library routines
    o3, s3 = oracle.prefill_fused(qb, kb, tok.v, tok.g, tok.beta, None, None, cu, init, scale=0.25, qk_l2norm=True)
    q64 = bf16_bits_to_f32(qb).astype(np.float64)
    k64 = bf16_bits_to_f32(kb).astype(np.float64)
    qn = 0.25 * q64 / np.sqrt(np.einsum("thd,thd->th", q64, q64) + 1e-6)[..., None]
    kn = k64 / np.sqrt(np.einsum("thd,thd->th", k64, k64) + 1e-6)[..., None]
    for n, (t0, t1) in enumerate([(0, 29), (29, 40)]):
        for h in range(4):
            v64 = bf16_bits_to_f32(tok.v[t0:t1, h]).astype(np.float64)
            g64, b64 = tok.g[t0:t1, h].astype(np.float64), tok.beta[t0:t1, h].astype(np.float64)
            S0 = init[n, h].astype(np.float64)
            for form in (R.paper_form, lambda *a: R.chunked(*a, C=8)):
                ro, rs = form(qn[t0:t1, h // 2], kn[t0:t1, h // 2], v64, g64, b64, S0)
                np.testing.assert_allclose(o3[t0:t1, h], ro, rtol=1e-10, atol=1e-13)
                np.testing.assert_allclose(s3[n, h], rs, rtol=1e-10, atol=1e-13)
    # the norms really were far from 1: without normalisation the result differs grossly
    assert rel_fro(0.25 * o0, o3) > 0.1
    # (4) invariance: rescaling q and k per token by powers of two changes nothing but the 1e-6 term
    o4, s4 = oracle.prefill_fused(tok.q, tok.k, tok.v, tok.g, tok.beta, None, None, cu, init, scale=0.25, qk_l2norm=True)
    # tok.k has norm 1 and tok.q norm 1/4: the 1e-6 under the root moves the unit vectors by < 1e-5 relative
    assert rel_fro(o3, o4) < 2e-4 and rel_fro(s3, s4) < 2e-4
    big_k = f32_to_bf16_bits(bf16_bits_to_f32(tok.k) * np.float32(1024.0))
    big_q = f32_to_bf16_bits(bf16_bits_to_f32(tok.q) * np.float32(4096.0))
    big_k2 = f32_to_bf16_bits(bf16_bits_to_f32(big_k) * pw_k)
    big_q2 = f32_to_bf16_bits(bf16_bits_to_f32(big_q) * pw_q)
    o5, s5 = oracle.prefill_fused(big_q, big_k, tok.v, tok.g, tok.beta, None, None, cu, init, scale=0.25, qk_l2norm=True)
    o6, s6 = oracle.prefill_fused(big_q2, big_k2, tok.v, tok.g, tok.beta, None, None, cu, init, scale=0.25, qk_l2norm=True)
    assert rel_fro(o6, o5) < 1e-10 and rel_fro(s6, s5) < 1e-10   # 1e-6 against squared norms >= 6e4
    # (5) recall with one-hot keys of magnitude 3: normalised they are unit vectors, so with g = 0, beta = 1
    #     the state returns v_s for q = k_s exactly (up to the 1e-6 under the root: 1 - 9/(9+1e-6) ~ 1e-7)
    T, dk, dv = 6, 8, 5
    idx = np.array([2, 5, 0, 7, 3, 5])                      # key 5 is written twice: the second write wins
    kk = np.zeros((T, 1, dk), np.float32)
    kk[np.arange(T), 0, idx] = 3.0
    vv = rng.standard_normal((T, 1, dv)).astype(np.float32)
    vb, v_exact = round_bf16(vv)
    oo, ss = oracle.prefill_fused(f32_to_bf16_bits(kk), f32_to_bf16_bits(kk), vb, np.zeros((T, 1), np.float32),
                                  np.ones((T, 1), np.float32), None, None, make_cu_seqlens([T]), None,
                                  scale=2.0, qk_l2norm=True)
    np.testing.assert_allclose(oo[:, 0], 2.0 * v_exact[:, 0], rtol=1e-6, atol=1e-12)   # o_t = scale * v_t
    last = {int(j): t for t, j in enumerate(idx)}
    for j, t in last.items():
        np.testing.assert_allclose(ss[0, 0][:, j], v_exact[t, 0], rtol=1e-6, atol=1e-12)
    # (6) raw gates and the front end together; decode form = one-token sequences
    from gdn_inputs import make_raw_gates
    a, b, A_log, dt_bias = make_raw_gates(40, 4, seed=200)
    o7, s7 = oracle.prefill_fused(qb, kb, tok.v, a, b, A_log, dt_bias, cu, init, scale=0.25, qk_l2norm=True)
    o8, s8 = oracle.prefill_fused(qb, kb, tok.v, a, b, A_log, dt_bias, cu, init, scale=1.0, qk_l2norm=True)
    np.testing.assert_allclose(o7, 0.25 * o8, rtol=1e-13, atol=1e-300)
    x = a.astype(np.float64) + dt_bias.astype(np.float64)[None, :]
    g64 = (-np.exp(A_log.astype(np.float64))[None, :] * np.logaddexp(0.0, x)).astype(np.float32)
    beta64 = (1.0 / (1.0 + np.exp(-b.astype(np.float64)))).astype(np.float32)
    o9, s9 = oracle.prefill_fused(qb, kb, tok.v, g64, beta64, None, None, cu, init, scale=0.25, qk_l2norm=True)
    assert rel_fro(o7, o9) < 1e-6 and rel_fro(s7, s9) < 1e-6
    st = make_state(40, 4, 16, 6, seed=201, sd=0.3)
    od, sd = oracle.decode_fused(qb, kb, tok.v, a, b, A_log, dt_bias, st, scale=0.25, qk_l2norm=True)
    op, sp = oracle.prefill_fused(qb, kb, tok.v, a, b, A_log, dt_bias, make_cu_seqlens([1] * 40), st, scale=0.25, qk_l2norm=True)
    np.testing.assert_array_equal(od, op)
    np.testing.assert_array_equal(sd, sp)
