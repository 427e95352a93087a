"""Pins for the CPU oracle: what the paper's equations and plain linear algebra fix.

Each test is chosen so that a plausible slip in the oracle (a dropped decay, a
wrong sign, S k versus S^T k, parents walked in the wrong direction, the output
read before the update) fails at least one of them.  None of the expected
values below comes from the oracle itself or from the CUDA library.
"""
import itertools
import json
from pathlib import Path

import numpy as np
import pytest

import oracle
from oracle import evaluators as ev

GOLDEN = Path(__file__).parent / "golden"


def _rand_steps(rng, T, W, H, dk, dv, unit_k=True):
    steps = []
    for _ in range(T):
        k = rng.standard_normal((W, H, dk))
        if unit_k:
            k /= np.linalg.norm(k, axis=-1, keepdims=True)
        steps.append({"k": k.astype(np.float32), "v": rng.standard_normal((W, H, dv)).astype(np.float32),
                      "alpha": rng.uniform(0.5, 1.0, (W, H)).astype(np.float32),
                      "beta": rng.uniform(0.0, 1.0, (W, H)).astype(np.float32)})
    return steps


def _rand_parents(rng, T, W):
    return [None] + [rng.integers(0, W, W).astype(np.int32) for _ in range(1, T)]


def _chain_of(steps, parents, b, h):
    """Records of unit (b, h), oldest first, by walking parent pointers (test-local)."""
    T = len(steps)
    idx, cur = [0] * T, b
    for t in range(T - 1, -1, -1):
        idx[t] = cur
        if t > 0:
            cur = int(parents[t][cur])
    return [(steps[t]["k"][idx[t], h], steps[t]["v"][idx[t], h], float(steps[t]["alpha"][idx[t], h]),
             float(steps[t]["beta"][idx[t], h])) for t in range(T)], idx


# --- hand-worked examples ------------------------------------------------------------------
@pytest.mark.parametrize("ex", json.loads((GOLDEN / "hand_examples.json").read_text())["examples"],
                         ids=lambda e: e["name"])
def test_hand_examples(ex):
    S0 = np.array(ex["S0"], dtype=np.float32)[None]            # one head
    T = len(ex["chain"])
    steps = [{"k": np.array(r["k"], np.float32)[None, None], "v": np.array(r["v"], np.float32)[None, None],
              "alpha": np.array([[r["alpha"]]], np.float32), "beta": np.array([[r["beta"]]], np.float32)}
             for r in ex["chain"]]
    parents = [None] + [np.zeros(1, np.int32)] * (T - 1)
    q = np.array(ex["q"], np.float32)[None, None]
    out = oracle.decode(S0, steps, parents, q)
    np.testing.assert_allclose(out[0, 0], ex["o"], rtol=0, atol=1e-14)
    # the intermediate states: read column e_j of S_t with q = e_j after t+1 records
    dv, dk = S0.shape[1:]
    for t, St in enumerate(ex["states"]):
        got = np.stack([oracle.decode(S0, steps[: t + 1], parents[: t + 1],
                                      np.eye(dk, dtype=np.float32)[j][None, None])[0, 0] for j in range(dk)], 1)
        np.testing.assert_allclose(got, np.array(St), rtol=0, atol=1e-14)
    # the other two evaluators on the same numbers
    chain = [(np.array(r["k"]), np.array(r["v"]), r["alpha"], r["beta"]) for r in ex["chain"]]
    np.testing.assert_allclose(ev.forward_projection_replay(ex["S0"], chain, ex["q"]), ex["o"], atol=1e-14)
    np.testing.assert_allclose(ev.backward_fold(ex["S0"], chain, ex["q"]), ex["o"], atol=1e-14)


# --- invariants ----------------------------------------------------------------------------
def test_alpha1_beta0_is_plain_matvec():
    rng = np.random.default_rng(1)
    T, W, H, dk, dv = 3, 5, 2, 7, 4
    steps = _rand_steps(rng, T, W, H, dk, dv)
    for s in steps:
        s["alpha"][:] = 1.0
        s["beta"][:] = 0.0
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    q = rng.standard_normal((W, H, dk)).astype(np.float32)
    out = oracle.decode(S0, steps, _rand_parents(rng, T, W), q)
    want = np.einsum("hij,bhj->bhi", S0.astype(np.float64), q.astype(np.float64))
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-13)


def test_beta1_unit_key_overwrites_value():
    """beta_t = 1 and |k_t| = 1  =>  S_t k_t = v_t, whatever alpha_t and the parent state."""
    rng = np.random.default_rng(2)
    T, W, H, dk, dv = 3, 4, 2, 8, 5
    steps = _rand_steps(rng, T, W, H, dk, dv)
    last = steps[-1]
    k = np.zeros((W, H, dk), np.float32)           # exactly unit in fp32: four entries of +-0.5
    for b in range(W):
        for h in range(H):
            pos = rng.choice(dk, 4, replace=False)
            k[b, h, pos] = rng.choice([-0.5, 0.5], 4)
    last["k"], last["beta"][:] = k, 1.0
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    out = oracle.decode(S0, steps, _rand_parents(rng, T, W), k)     # q = k_t
    np.testing.assert_allclose(out, last["v"].astype(np.float64), rtol=0, atol=1e-13)


def test_shared_chain_gives_identical_outputs():
    rng = np.random.default_rng(3)
    T, W, H, dk, dv = 3, 6, 2, 8, 8
    steps = _rand_steps(rng, T, W, H, dk, dv)
    parents = [None, rng.integers(0, W, W).astype(np.int32), np.full(W, 2, np.int32)]
    for name in ("k", "v", "alpha", "beta"):
        steps[-1][name][:] = steps[-1][name][0]      # same new token on every beam
    q = np.repeat(rng.standard_normal((1, H, dk)).astype(np.float32), W, 0)
    out = oracle.decode(rng.standard_normal((H, dv, dk)).astype(np.float32), steps, parents, q)
    for b in range(1, W):
        assert np.array_equal(out[b], out[0])


def test_output_depends_on_chain_not_on_siblings():
    """Changing a record no chain refers to changes nothing; changing one on the chain does."""
    rng = np.random.default_rng(4)
    T, W, H, dk, dv = 3, 4, 1, 6, 6
    steps = _rand_steps(rng, T, W, H, dk, dv)
    parents = [None, np.array([1, 1, 3, 3], np.int32), np.array([0, 0, 1, 1], np.int32)]
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    q = rng.standard_normal((W, H, dk)).astype(np.float32)
    base = oracle.decode(S0, steps, parents, q)
    steps[0]["v"][0] += 1.0                          # beam 0 of call 0 is nobody's ancestor
    steps[1]["v"][2] += 1.0                          # beam 2 of call 1 is nobody's parent
    assert np.array_equal(oracle.decode(S0, steps, parents, q), base)
    steps[0]["v"][1] += 1.0                          # ancestor of every beam
    assert np.all(np.abs(oracle.decode(S0, steps, parents, q) - base).max(axis=-1) > 1e-3)


# --- closed form: distinct one-hot keys ------------------------------------------------------
def test_one_hot_keys_closed_form():
    """k_j = e_{i_j}: column i_j becomes alpha(1-beta) col + beta v, every other column is scaled by alpha."""
    rng = np.random.default_rng(5)
    T, dk, dv = 4, 6, 3
    S0 = rng.standard_normal((1, dv, dk)).astype(np.float32)
    cols = rng.permutation(dk)[:T]
    steps, S = [], S0[0].astype(np.float64).copy()
    for j in range(T):
        k = np.zeros(dk, np.float32)
        k[cols[j]] = 1.0
        v = rng.standard_normal(dv).astype(np.float32)
        a, b = np.float32(rng.uniform(0.5, 1)), np.float32(rng.uniform(0, 1))
        steps.append({"k": k[None, None], "v": v[None, None], "alpha": np.array([[a]]), "beta": np.array([[b]])})
        keep = S[:, cols[j]].copy()
        S *= float(a)
        S[:, cols[j]] = float(a) * (1.0 - float(b)) * keep + float(b) * v.astype(np.float64)
    q = rng.standard_normal((1, 1, dk)).astype(np.float32)
    out = oracle.decode(S0, steps, [None] + [np.zeros(1, np.int32)] * (T - 1), q)
    np.testing.assert_allclose(out[0, 0], S @ q[0, 0].astype(np.float64), rtol=0, atol=1e-13)


# --- brute force: dense operator products over every lineage of a tiny beam ----------------------
def _dense_state(S0, chain):
    """S_T = S_0 prod_j A_j + sum_j beta_j v_j k_j^T prod_{i>j} A_i with A_j = alpha_j (I - beta_j k_j k_j^T)."""
    dk = S0.shape[1]
    A = [a * (np.eye(dk) - b * np.outer(k, k)) for (k, v, a, b) in chain]
    def tail(j):
        P = np.eye(dk)
        for i in range(j, len(chain)):
            P = P @ A[i]
        return P
    S = S0 @ tail(0)
    for j, (k, v, a, b) in enumerate(chain):
        S = S + b * np.outer(v, k) @ tail(j + 1)
    return S


@pytest.mark.parametrize("W,T", [(2, 3), (3, 3)])
def test_brute_force_every_parent_map(W, T):
    rng = np.random.default_rng(6)
    H, dk, dv = 2, 5, 3
    steps = _rand_steps(rng, T, W, H, dk, dv, unit_k=False)
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    q = rng.standard_normal((W, H, dk)).astype(np.float32)
    maps = list(itertools.product(range(W), repeat=W))
    seen = set()
    for pm in itertools.product(maps, repeat=T - 1):
        parents = [None] + [np.array(p, np.int32) for p in pm]
        out, chains = oracle.decode(S0, steps, parents, q, return_chains=True)
        chains = chains.reshape(W, H, T)
        for b in range(W):
            for h in range(H):
                chain, idx = _chain_of(steps, parents, b, h)
                assert list(chains[b, h]) == idx
                seen.add(tuple(idx))
                chain64 = [(k.astype(np.float64), v.astype(np.float64), a, bb) for (k, v, a, bb) in chain]
                S = _dense_state(S0[h].astype(np.float64), chain64)
                np.testing.assert_allclose(out[b, h], S @ q[b, h].astype(np.float64), rtol=0, atol=1e-12)
    assert len(seen) == W ** T            # every lineage (b_0, ..., b_{T-1}) occurred


# --- three evaluators agree; rectangular state ------------------------------------------------
@pytest.mark.parametrize("dk,dv,T", [(16, 16, 6), (12, 20, 4), (32, 8, 1), (8, 8, 0)])
def test_three_evaluators_agree(dk, dv, T):
    rng = np.random.default_rng(7)
    W, H = 5, 3
    steps = _rand_steps(rng, T, W, H, dk, dv)
    parents = _rand_parents(rng, T, W)
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    q = rng.standard_normal((W, H, dk)).astype(np.float32)
    out = oracle.decode(S0, steps, parents, q)
    for b in range(W):
        for h in range(H):
            chain, _ = (_chain_of(steps, parents, b, h) if T else ([], None))
            fwd = ev.forward_projection_replay(S0[h], chain, q[b, h])
            bwd = ev.backward_fold(S0[h], chain, q[b, h])
            scale = max(np.linalg.norm(out[b, h]), 1e-30)
            assert np.linalg.norm(fwd - out[b, h]) / scale < 1e-12
            assert np.linalg.norm(bwd - out[b, h]) / scale < 1e-12


def test_selected_units_match_full_run():
    rng = np.random.default_rng(8)
    T, W, H, dk, dv = 3, 7, 3, 8, 6
    steps, parents = _rand_steps(rng, T, W, H, dk, dv), _rand_parents(rng, T, W)
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    q = rng.standard_normal((W, H, dk)).astype(np.float32)
    full = oracle.decode(S0, steps, parents, q)
    beams, heads = np.array([6, 0, 3, 3]), np.array([2, 1, 0, 2])
    sel = oracle.decode(S0, steps, parents, q, sel=(beams, heads), nthreads=1)
    for i in range(4):
        assert np.array_equal(sel[i], full[beams[i], heads[i]])


# --- linearity ----------------------------------------------------------------------------
def test_linearity_in_q_S0_and_v():
    rng = np.random.default_rng(9)
    T, W, H, dk, dv = 3, 4, 2, 8, 8
    steps, parents = _rand_steps(rng, T, W, H, dk, dv), _rand_parents(rng, T, W)
    # fp32 inputs whose sums are exact in fp32 (small dyadic rationals)
    def dy(shape):
        return (rng.integers(-64, 65, shape) / 64.0).astype(np.float32)
    S0a, S0b, q1, q2 = dy((H, dv, dk)), dy((H, dv, dk)), dy((W, H, dk)), dy((W, H, dk))
    f = lambda S0, q: oracle.decode(S0, steps, parents, q)
    np.testing.assert_allclose(f(S0a, q1 + q2), f(S0a, q1) + f(S0a, q2), atol=1e-12)
    zero = np.zeros_like(S0a)
    # o = S_0 r + corr: affine in S_0 (the records' own contribution does not scale with S_0)
    np.testing.assert_allclose(f(S0a + S0b, q1) + f(zero, q1), f(S0a, q1) + f(S0b, q1), atol=1e-12)
    base = f(zero, q1)                                  # S0 = 0: only the records' contribution
    for s in steps:
        s["v"] = s["v"] * np.float32(2.0)
    np.testing.assert_allclose(f(zero, q1), 2.0 * base, atol=1e-12)


# --- ancestry (Eq. 5) against the linked walk -------------------------------------------------
def _chains(parents, W, T):
    H, dk, dv = 1, 2, 2
    steps = [{"k": np.zeros((W, H, dk), np.float32), "v": np.zeros((W, H, dv), np.float32),
              "alpha": np.ones((W, H), np.float32), "beta": np.zeros((W, H), np.float32)} for _ in range(T)]
    _, chains = oracle.decode(np.zeros((H, dv, dk), np.float32), steps, parents,
                              np.zeros((W, H, dk), np.float32), return_chains=True)
    return chains


def test_ancestry_table_equals_pointer_walk():
    rng = np.random.default_rng(10)
    W, T = 9, 5
    parents = _rand_parents(rng, T, W)
    assert np.array_equal(_chains(parents, W, T), ev.ancestry_table(parents, [W] * T))


def test_ancestry_special_parent_maps():
    W, T = 6, 4
    ident = [None] + [np.arange(W, dtype=np.int32)] * (T - 1)
    assert np.array_equal(_chains(ident, W, T), np.repeat(np.arange(W)[:, None], T, 1))
    const = [None] + [np.full(W, 4, np.int32)] * (T - 1)
    c = _chains(const, W, T)
    assert np.all(c[:, :-1] == 4) and np.array_equal(c[:, -1], np.arange(W))
    rng = np.random.default_rng(11)
    perms = [None] + [rng.permutation(W).astype(np.int32) for _ in range(T - 1)]
    c = _chains(perms, W, T)
    for b in range(W):                                    # composition of permutations
        assert c[b, 2] == perms[3][b] and c[b, 1] == perms[2][perms[3][b]] and c[b, 0] == perms[1][perms[2][perms[3][b]]]
    # a beam nobody selects appears in no row
    p = [None, np.array([0, 0, 2, 2, 4, 4], np.int32), np.array([1, 1, 1, 3, 3, 5], np.int32)]
    c = _chains(p, W, 3)
    assert set(c[:, 1]) == {1, 3, 5} and set(c[:, 0]) == {0, 2, 4}


def test_varying_beam_width_and_bad_parent():
    rng = np.random.default_rng(12)
    H, dk, dv, Ws = 1, 4, 4, [3, 5, 2]
    steps = []
    for W in Ws:
        steps += _rand_steps(rng, 1, W, H, dk, dv)
    parents = [None, rng.integers(0, 3, 5).astype(np.int32), rng.integers(0, 5, 2).astype(np.int32)]
    S0 = rng.standard_normal((H, dv, dk)).astype(np.float32)
    q = rng.standard_normal((2, H, dk)).astype(np.float32)
    out = oracle.decode(S0, steps, parents, q)
    for b in range(2):
        chain, _ = _chain_of(steps, parents, b, 0)
        np.testing.assert_allclose(out[b, 0], ev.backward_fold(S0[0], chain, q[b, 0]), atol=1e-12)
    parents[2] = np.array([0, 5], np.int32)               # 5 is outside a beam of width 5
    with pytest.raises(ValueError):
        oracle.decode(S0, steps, parents, q)


# --- prefill (how S_0 is defined) ---------------------------------------------------------
def test_prefill_orthonormal_keys_is_associative_memory():
    """alpha = beta = 1 with orthonormal keys: S = sum_i v_i k_i^T and S k_i = v_i."""
    rng = np.random.default_rng(13)
    H, dk, dv, N = 2, 8, 5, 6
    k = np.zeros((N, H, dk), np.float32)
    for h in range(H):
        cols = rng.permutation(dk)[:N]
        for i in range(N):
            k[i, h, cols[i]] = rng.choice([-1.0, 1.0])
    v = rng.standard_normal((N, H, dv)).astype(np.float32)
    one = np.ones((N, H), np.float32)
    S = oracle.prefill(k, v, one, one)
    want = np.einsum("nhi,nhj->hij", v.astype(np.float64), k.astype(np.float64))
    np.testing.assert_allclose(S, want, atol=1e-14)
    np.testing.assert_allclose(np.einsum("hij,nhj->nhi", S, k.astype(np.float64)), v, atol=1e-14)


def test_prefill_decay_only_and_single_token():
    rng = np.random.default_rng(14)
    H, dk, dv, N = 1, 4, 3, 5
    k = rng.standard_normal((N, H, dk)).astype(np.float32)
    v = rng.standard_normal((N, H, dv)).astype(np.float32)
    a = rng.uniform(0.5, 1, (N, H)).astype(np.float32)
    assert np.all(oracle.prefill(k, v, a, np.zeros((N, H), np.float32)) == 0.0)     # beta = 0: nothing written
    b = rng.uniform(0, 1, (N, H)).astype(np.float32)
    S1 = oracle.prefill(k[:1], v[:1], a[:1], b[:1])                                   # from zero: S = beta v k^T
    np.testing.assert_allclose(S1[0], float(b[0, 0]) * np.outer(v[0, 0].astype(np.float64), k[0, 0].astype(np.float64)), atol=1e-15)
    # with a one-hot first key and beta = 0 afterwards the state only decays: S_N = (prod alpha) S_1
    bb = b.copy()
    bb[1:] = 0.0
    SN = oracle.prefill(k, v, a, bb)
    np.testing.assert_allclose(SN, np.prod(a[1:].astype(np.float64)) * S1, rtol=1e-14)


def test_prefill_then_decode_equals_one_long_chain():
    rng = np.random.default_rng(15)
    H, dk, dv, N, T = 2, 6, 4, 5, 2
    tok = _rand_steps(rng, N + T, 1, H, dk, dv)
    cat = lambda n, lo, hi: np.concatenate([tok[i][n] for i in range(lo, hi)], 0)
    S0 = oracle.prefill(cat("k", 0, N), cat("v", 0, N), cat("alpha", 0, N), cat("beta", 0, N))
    q = rng.standard_normal((1, H, dk)).astype(np.float32)
    zero = np.zeros((H, dv, dk), np.float32)
    ident = lambda n: [None] + [np.zeros(1, np.int32)] * (n - 1)
    long = oracle.decode(zero, tok, ident(N + T), q)
    # S0 is handed over in fp32 (as the store holds it), so compare at fp32 resolution
    short = oracle.decode(S0.astype(np.float32), tok[N:], ident(T), q)
    np.testing.assert_allclose(short, long, rtol=0, atol=5e-6)


def test_grouped_value_heads_equal_one_single_head_run_per_value_head():
    """Value head j of a grouped layer is an ordinary single-head layer with key head j // g's queries and keys:
    the grouped evaluation must equal Hv separate one-head runs (each through the pinned ungrouped routine)."""
    rng = np.random.default_rng(21)
    Hk, g, dk, dv, W, T = 2, 3, 8, 6, 5, 3
    Hv = Hk * g
    S0 = rng.normal(size=(Hv, dv, dk))
    steps = [{"k": rng.normal(size=(W, Hk, dk)), "v": rng.normal(size=(W, Hv, dv)),
              "alpha": rng.uniform(0.9, 1.0, size=(W, Hv)), "beta": rng.uniform(0.1, 0.9, size=(W, Hv))} for _ in range(T)]
    parents = [None] + [rng.integers(0, W, W) for _ in range(T - 1)]
    q = rng.normal(size=(W, Hk, dk))
    got = oracle.decode_grouped(S0, steps, parents, q)
    for j in range(Hv):
        one = [{"k": s["k"][:, j // g:j // g + 1], "v": s["v"][:, j:j + 1], "alpha": s["alpha"][:, j:j + 1],
                "beta": s["beta"][:, j:j + 1]} for s in steps]
        want = oracle.decode(S0[j:j + 1], one, parents, q[:, j // g:j // g + 1])
        # inputs pass through fp32 on the way in, identically on both sides
        assert np.allclose(got[:, j], want[:, 0], rtol=1e-12, atol=1e-12)
    # g = 1 is the ungrouped routine itself
    steps1 = [dict(s, v=s["v"][:, :Hk], alpha=s["alpha"][:, :Hk], beta=s["beta"][:, :Hk]) for s in steps]
    assert np.array_equal(oracle.decode_grouped(S0[:Hk], steps1, parents, q), oracle.decode(S0[:Hk], steps1, parents, q))
