"""Pins for the CPU oracle: closed forms, invariants, brute force and library special cases.

The paper prints no worked numeric example for this path, so the oracle is pinned by what
the mathematics fixes.  Each pin is chosen so that a plausible slip in the oracle (dropped
bias, transposed weight, sum instead of mean, wrong tie-break, missing scale, swapped key
segments) makes it fail.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2601_21896_b200 import workloads as wl

bf = wl.f32_to_bf16_bits
f32 = wl.bf16_bits_to_f32


def _bits(x):
    return bf(np.asarray(x, dtype=np.float32))


# ----------------------------------------------------------------- golden constants
def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")
    out = {}
    for line in open(path):
        line = line.split("#")[0].split()
        if line:
            out[line[0]] = [int(v) for v in line[1:]]
    return out


def test_workload_geometry_matches_paper_constants():
    g = _golden()
    assert wl.TOKENS_PER_FRAME == g["tokens_per_frame"][0]
    assert wl.CHUNK_TOKENS == g["chunk_tokens"][0] == 3 * g["tokens_per_frame"][0]
    w = wl.wan13b_layer()
    assert (w.n_heads, w.d_head, w.d_model) == (g["n_heads"][0], g["d_head"][0], g["d_model"][0])
    assert w.Lq[0] == g["chunk_tokens"][0]
    p = wl.paper_native()
    assert p.budget[0] == g["cache_tokens_full_model"][0]
    assert all(c % g["tokens_per_frame"][0] == 0 for c in g["cache_ablation"])
    assert g["smlp_dims"] == [3 * g["d_model"][0], 1024, g["n_heads"][0]]


# ----------------------------------------------------------------------------- score
def test_score_hand_computed_token():
    # x = (1, 2); W1 = [[1, .5], [-1, .25]], b1 = (.5, 0) -> a = (2.5, -0.5)
    # W2 = [1, 2], b2 = .25.  SiLU: 2.5 s(2.5) + 2 (-.5 s(-.5)) + .25 with the tabulated
    # logistic values s(2.5) = 0.92414182, s(-0.5) = 0.37754067; GELU with the normal cdf
    # Phi(2.5) = 0.99379033, Phi(-0.5) = 0.30853754.
    X = _bits([[1.0, 2.0]])
    w1 = _bits([[1.0, 0.5], [-1.0, 0.25]]); b1 = _bits([0.5, 0.0])
    w2 = _bits([[1.0, 2.0]]); b2 = _bits([0.25])
    s_silu = oracle.score(X, w1, b1, w2, b2, act=wl.ACT_SILU)[0]
    s_gelu = oracle.score(X, w1, b1, w2, b2, act=wl.ACT_GELU)[0]
    assert abs(s_silu - 2.1828138811) < 1e-6
    assert abs(s_gelu - 2.4259382980) < 1e-6
    # final sigmoid of the GELU value: 1 / (1 + e^-2.4259383) = 1 / 1.0883951 = 0.918784
    s_sig = oracle.score(X, w1, b1, w2, b2, act=wl.ACT_GELU, final=wl.FINAL_SIGMOID)[0]
    assert abs(s_sig - 0.9187840) < 1e-6


def test_score_zero_preactivation_and_sigmoid_half():
    rng = np.random.default_rng(1)
    X = bf(rng.standard_normal((5, 16)).astype(np.float32))
    w1 = np.zeros((8, 16), np.uint16)
    w2 = bf(rng.standard_normal((3, 8)).astype(np.float32))
    for act in (wl.ACT_GELU, wl.ACT_SILU):
        s = oracle.score(X, w1, None, w2, None, act=act)       # act(0) = 0 -> score 0
        assert np.all(s == 0.0)
        s = oracle.score(X, w1, None, w2, None, act=act, final=wl.FINAL_SIGMOID)
        assert np.all(s == 0.5)                                  # sigma(0) = 1/2
    # W1 = 0 with biases: every token gets mean_o(W2 act(b1) + b2), independent of x
    b1 = _bits(np.linspace(-2, 2, 8)); b2 = _bits([0.5, -1.0, 2.0])
    s = oracle.score(X, w1, b1, w2, b2, act=wl.ACT_SILU)
    b1f = f32(b1).astype(np.float64)
    h = b1f / (1 + np.exp(-b1f))
    want = np.mean(f32(w2).astype(np.float64) @ h + f32(b2))
    assert np.allclose(s, want, atol=1e-6) and np.all(s == s[0])


def test_score_mean_over_outputs_equals_single_output():
    # Appendix A: the 12 outputs are averaged.  12 identical output rows == one output.
    rng = np.random.default_rng(2)
    X = bf(rng.standard_normal((7, 24)).astype(np.float32))
    w1 = bf(rng.standard_normal((10, 24)).astype(np.float32) / 5)
    b1 = bf(rng.standard_normal(10).astype(np.float32))
    w2 = bf(rng.standard_normal((1, 10)).astype(np.float32)); b2 = _bits([0.75])
    one = oracle.score(X, w1, b1, w2, b2, act=wl.ACT_SILU)
    twelve = oracle.score(X, w1, b1, np.repeat(w2, 12, 0), np.repeat(b2, 12), act=wl.ACT_SILU)
    assert np.allclose(one, twelve, atol=1e-6)
    # linear in (W2, b2): doubling both doubles the score (power of two is exact in bf16)
    dbl = oracle.score(X, w1, b1, bf(2 * f32(w2)), bf(2 * f32(b2)), act=wl.ACT_SILU)
    assert np.allclose(dbl, 2 * one, atol=1e-6)


@pytest.mark.parametrize("act", [wl.ACT_GELU, wl.ACT_SILU])
@pytest.mark.parametrize("final", [wl.FINAL_NONE, wl.FINAL_SIGMOID])
def test_score_against_torch_float64_linear(act, final):
    rng = np.random.default_rng(3)
    n, d_in, d_h, d_o = 33, 48, 20, 12
    X = bf(rng.standard_normal((n, d_in)).astype(np.float32))
    w1 = bf(rng.standard_normal((d_h, d_in)).astype(np.float32) / 4)
    b1 = bf(rng.standard_normal(d_h).astype(np.float32))
    w2 = bf(rng.standard_normal((d_o, d_h)).astype(np.float32) / 4)
    b2 = bf(rng.standard_normal(d_o).astype(np.float32))
    t = lambda a: torch.from_numpy(f32(a)).double()
    h = torch.nn.functional.linear(t(X), t(w1), t(b1))
    h = torch.nn.functional.gelu(h) if act == wl.ACT_GELU else torch.nn.functional.silu(h)
    y = torch.nn.functional.linear(h, t(w2), t(b2)).mean(dim=1)
    if final:
        y = torch.sigmoid(y)
    got = oracle.score(X, w1, b1, w2, b2, act=act, final=final)
    assert np.allclose(got, y.numpy(), atol=1e-6, rtol=1e-6)


# ---------------------------------------------------------------------------- select


def brute_select(scores, n_sink, n_recent, budget):
    """O(M^2) rank counting: candidate c is kept iff fewer than k candidates beat it."""
    T = len(scores)
    if T <= budget:
        return list(range(T))
    nr = min(n_recent, budget)
    ns = min(n_sink, budget - nr)
    k = budget - ns - nr
    cand = list(range(ns, T - nr))

    def beats(a, b):
        sa, sb = scores[a], scores[b]
        na, nb = math.isnan(sa), math.isnan(sb)
        if na or nb:
            if na and nb:
                return a < b
            return nb
        if sa != sb:
            return sa > sb
        return a < b
    kept = [c for c in cand if sum(beats(o, c) for o in cand) < k]
    return sorted(list(range(ns)) + kept + list(range(T - nr, T)))


@pytest.mark.parametrize("kind", ["normal", "ties", "equal", "saturated", "heavy", "signed_zero"])
def test_select_equals_brute_force_on_tiny_inputs(kind):
    for seed in range(12):
        T = 8 + 5 * seed
        s = wl.random_scores(T, seed=seed, kind=kind, tag=T)
        for (ns, nr, B) in [(0, 0, T // 2), (2, 3, T // 2 + 2), (3, 0, 5), (0, 4, 4), (2, 2, 4),
                            (1, 1, T - 1), (4, 4, 3), (T, T, T // 3), (0, 0, 0), (1, 2, T),
                            (1, 2, T + 5)]:
            got = oracle.select(s, ns, nr, B)
            want = brute_select([float(v) for v in s], ns, nr, B)
            assert got.tolist() == want, (kind, seed, ns, nr, B)


def test_select_special_values_and_tiebreak():
    s = np.array([0.0, -0.0, 1.0, -np.inf, np.inf, np.nan, 1.0, -0.0, 0.0, np.nan], np.float32)
    # top-4 of all: inf(4), 1.0(2), 1.0(6), then the zeros tie -> lowest index 0
    assert oracle.select(s, 0, 0, 4).tolist() == [0, 2, 4, 6]
    # top-8: zeros 0,1,7,8 then -inf(3) ; NaN ranks last
    assert oracle.select(s, 0, 0, 8).tolist() == [0, 1, 2, 3, 4, 6, 7, 8]
    assert oracle.select(s, 0, 0, 9).tolist() == [0, 1, 2, 3, 4, 5, 6, 7, 8]
    # all equal -> lowest indices among candidates
    e = np.full(20, 0.25, np.float32)
    assert oracle.select(e, 2, 3, 9).tolist() == [0, 1, 2, 3, 4, 5, 17, 18, 19]


def test_select_invariants_at_paper_sizes():
    w = wl.wan13b_layer()
    T, B = w.T[0], w.budget[0]
    s = wl.random_scores(T, seed=5, kind="saturated")
    idx = oracle.select(s, w.n_sink, w.n_recent, B)
    assert len(idx) == B == 14040
    assert np.all(np.diff(idx) > 0) and idx[0] >= 0 and idx[-1] < T
    assert np.array_equal(idx[: w.n_sink], np.arange(w.n_sink))               # frame sink
    assert np.array_equal(idx[-w.n_recent:], np.arange(T - w.n_recent, T))     # recent window
    mid = idx[w.n_sink: B - w.n_recent]
    assert len(mid) == 7800
    rejected = np.setdiff1d(np.arange(w.n_sink, T - w.n_recent), mid)
    assert s[mid].min() >= s[rejected].max()
    # among the boundary ties the lower indices are the ones kept
    thr = s[mid].min()
    tie_kept = mid[s[mid] == thr]; tie_rej = rejected[s[rejected] == thr]
    if len(tie_rej):
        assert tie_kept.max() < tie_rej.min()
    # a strictly increasing map that makes no new ties leaves the selection unchanged
    s2 = wl.random_scores(T, seed=6, kind="normal")
    a = oracle.select(s2, w.n_sink, w.n_recent, B)
    b = oracle.select((s2.astype(np.float64) * 2.0 + 8.0).astype(np.float32), w.n_sink, w.n_recent, B)
    assert np.array_equal(a, b)
    with pytest.raises(ValueError):
        oracle.select(s, -1, 0, 5)


# --------------------------------------------------------------------------- compact
def test_compact_identity_and_elementwise():
    rng = np.random.default_rng(7)
    K = rng.integers(0, 65536, size=(50, 3, 8), dtype=np.uint16)
    assert np.array_equal(oracle.compact(K, np.arange(50, dtype=np.int32)), K)
    idx = np.array([0, 3, 4, 17, 49], np.int32)
    out = oracle.compact(K, idx)
    for i, t in enumerate(idx):
        assert np.array_equal(out[i], K[t])
    SL = rng.standard_normal(50).astype(np.float32)
    assert np.array_equal(oracle.compact(SL, idx), SL[idx])
    # Algorithm 2: SL <- Select(SL; ids) stays aligned, so re-selecting with the same budget
    # on the compacted list keeps everything
    assert oracle.select(oracle.compact(SL, idx), 1, 1, len(idx)).tolist() == list(range(len(idx)))


# ------------------------------------------------------------------------- attention
def _rand_qkv(rng, Lq, Lk, N, D, scale=1.0):
    Q = bf(rng.standard_normal((Lq, N, D)).astype(np.float32) * scale)
    K = bf(rng.standard_normal((Lk, N, D)).astype(np.float32) * scale)
    V = bf(rng.standard_normal((Lk, N, D)).astype(np.float32))
    return Q, K, V


def _torch_sdpa(Q, K, V, scale=None):
    t = lambda a: torch.from_numpy(f32(a)).double().permute(1, 0, 2)    # [N, L, D]
    o = torch.nn.functional.scaled_dot_product_attention(t(Q), t(K), t(V), scale=scale)
    return o.permute(1, 0, 2).numpy()


def test_attention_full_cache_equals_library_softmax_attention():
    rng = np.random.default_rng(11)
    Q, K, V = _rand_qkv(rng, 19, 45, 3, 16)
    O, LSE = oracle.attention(Q, K, V, None, None)
    assert np.allclose(O, _torch_sdpa(Q, K, V), atol=1e-12)
    # default scale is 1/sqrt(D) (Sec. 3.2); an explicit other scale is honoured
    O2, _ = oracle.attention(Q, K, V, None, None, scale=0.3)
    assert np.allclose(O2, _torch_sdpa(Q, K, V, scale=0.3), atol=1e-12)
    assert not np.allclose(O, O2, atol=1e-3)
    # LSE against the definition via torch.logsumexp
    z = torch.einsum("qnd,knd->nqk", torch.from_numpy(f32(Q)).double(),
                     torch.from_numpy(f32(K)).double()) / math.sqrt(16)
    assert np.allclose(LSE, torch.logsumexp(z, dim=-1).numpy(), atol=1e-12)


def test_attention_two_segments_equal_concatenation_and_row_subset():
    rng = np.random.default_rng(12)
    Q, K, V = _rand_qkv(rng, 23, 40, 2, 8)
    Kq, Vq = K[29:], V[29:]
    O_cat, L_cat = oracle.attention(Q, K, V, None, None)
    O_seg, L_seg = oracle.attention(Q, K[:29], V[:29], Kq, Vq)
    assert np.allclose(O_cat, O_seg, atol=1e-13) and np.allclose(L_cat, L_seg, atol=1e-13)
    # swapping the V segments must change the result (segments are not interchangeable)
    O_bad, _ = oracle.attention(Q, K[:29], V[:29][::-1].copy(), Kq, Vq)
    assert not np.allclose(O_cat, O_bad, atol=1e-3)
    rows = [0, 5, 22]
    O_r, L_r = oracle.attention(Q, K[:29], V[:29], Kq, Vq, rows=rows)
    assert np.array_equal(O_r, O_seg[rows]) and np.array_equal(L_r, L_seg[:, rows])
    # merging two independent passes by their log-sum-exp equals one pass
    Oa, La = oracle.attention(Q, K[:29], V[:29], None, None)
    Ob, Lb = oracle.attention(Q, Kq, Vq, None, None)
    wa = np.exp(La - L_cat).T[:, :, None]; wb = np.exp(Lb - L_cat).T[:, :, None]
    assert np.allclose(wa * Oa + wb * Ob, O_cat, atol=1e-12)


def test_attention_closed_forms():
    rng = np.random.default_rng(13)
    Q, K, V = _rand_qkv(rng, 9, 30, 2, 8)
    ones = bf(np.ones((30, 2, 8), np.float32))
    O, _ = oracle.attention(Q, K, ones, None, None)
    assert np.allclose(O, 1.0, atol=1e-13)                         # softmax rows sum to one
    O, L = oracle.attention(Q, K[:1], V[:1], None, None)
    assert np.allclose(O, np.broadcast_to(f32(V[:1]), O.shape))    # one key -> its value
    Ksame = np.repeat(K[:1], 30, axis=0)
    O, _ = oracle.attention(Q, Ksame, V, None, None)
    assert np.allclose(O, f32(V).astype(np.float64).mean(0)[None], atol=1e-13)  # uniform weights
    perm = rng.permutation(30)
    Oa, _ = oracle.attention(Q, K, V, None, None)
    Ob, _ = oracle.attention(Q, K[perm], V[perm], None, None)
    assert np.allclose(Oa, Ob, atol=1e-13)                         # key order is irrelevant
    # huge logits stay finite thanks to the max subtraction
    Qb, Kb, Vb = _rand_qkv(rng, 4, 12, 1, 8, scale=300.0)
    O, L = oracle.attention(Qb, Kb, Vb, None, None)
    assert np.all(np.isfinite(O)) and np.all(np.isfinite(L))
    # a query equal to one key scaled up concentrates on that key
    big = f32(K[5:6]).astype(np.float32) * 512
    O, _ = oracle.attention(bf(big), K, V, None, None)
    assert np.allclose(O[0], f32(V[5]), atol=1e-6)


def test_pruning_to_full_budget_leaves_attention_unchanged():
    w = wl.tiny()
    d = wl.make_layer(w)
    s = oracle.score(d["K"].reshape(w.T[0], -1), d["w1"], d["b1"], d["w2"], d["b2"], w.act, w.final)
    idx_all = oracle.select(s, w.n_sink, w.n_recent, w.T[0])
    assert idx_all.tolist() == list(range(w.T[0]))
    Kc, Vc = oracle.compact(d["K"], idx_all), oracle.compact(d["V"], idx_all)
    rows = [0, 31, 63]
    O1, _ = oracle.attention(d["Q"], Kc, Vc, d["Kq"], d["Vq"], rows=rows)
    cat = lambda a, b: np.concatenate([a, b], 0)
    O2 = _torch_sdpa(d["Q"], cat(d["K"], d["Kq"]), cat(d["V"], d["Vq"]))[rows]
    assert np.allclose(O1, O2, atol=1e-12)
    # and the tiny config's budget: 4 sink + 64 recent + 60 by salience
    idx = oracle.select(s, w.n_sink, w.n_recent, w.budget[0])
    assert len(idx) == 128 and idx[:4].tolist() == [0, 1, 2, 3] and idx[-64] == 448


# ------------------------------------------------------------------------------- sse
def test_sse_against_dense_torch_softmax():
    rng = np.random.default_rng(21)
    L, N, D, LB = 24, 2, 8, 6
    Q = bf(rng.standard_normal((L, N, D)).astype(np.float32))
    K = bf(rng.standard_normal((L, N, D)).astype(np.float32))
    s, comp = oracle.sse(Q, K, LB)
    tq = torch.from_numpy(f32(Q)).double(); tk = torch.from_numpy(f32(K)).double()
    P = torch.softmax(torch.einsum("qnd,knd->nqk", tq, tk) / math.sqrt(D), dim=-1).numpy()
    qi = np.arange(L)[:, None]; kj = np.arange(L)[None, :]
    lo = (qi // LB) * LB; hi = lo + LB
    low = np.where(kj < lo, P, 0).max(1).mean(0)
    diag = np.where((kj >= lo) & (kj < hi), P, 0).max(1).mean(0)
    up = np.where(kj >= hi, P, 0).max(1).mean(0)
    assert np.allclose(comp, np.stack([low, diag, up]), atol=1e-13)
    want = np.where(kj[0] < LB, (diag + low) / 2,
                    np.where(kj[0] < L - LB, (up + diag + low) / 3, (diag + up) / 2))
    assert np.allclose(s, want, atol=1e-13)
    # first block has no earlier-block queries, last block no later-block queries
    assert np.all(comp[2, :LB] == 0) and np.all(comp[0, L - LB:] == 0)


def test_sse_uniform_attention_closed_form():
    # zero queries make every row of P uniform (1/L), so each class that has queries gives 1/L:
    # Eq. 5 then yields 1/L for every key, whichever case applies
    L, N, D, LB = 30, 3, 4, 7          # last block shorter than the others
    rng = np.random.default_rng(2)
    Q = np.zeros((L, N, D), np.uint16)
    K = bf(rng.standard_normal((L, N, D)).astype(np.float32))
    s, comp = oracle.sse(Q, K, LB)
    nb = -(-L // LB)
    kb = np.arange(L) // LB
    assert np.allclose(comp[0], np.where(kb < nb - 1, 1.0 / L, 0.0), atol=1e-15)   # later blocks exist
    assert np.allclose(comp[1], 1.0 / L, atol=1e-15)
    assert np.allclose(comp[2], np.where(kb > 0, 1.0 / L, 0.0), atol=1e-15)        # earlier blocks exist
    j = np.arange(L)
    want = np.where(j < LB, (1 / L + 1 / L) / 2, np.where(j < L - LB, 3 / L / 3, (1 / L + np.where(kb > 0, 1 / L, 0)) / 2))
    assert np.allclose(s, want, atol=1e-15)


def test_sse_brute_force_index_sets():
    # Eq. 4 written out with explicit index sets I_low(j) = {i | j < l(i)}, I_diag, I_up
    rng = np.random.default_rng(4)
    L, N, D, LB = 11, 2, 4, 4
    Q = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    K = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    scale = 0.37
    s, comp = oracle.sse(Q, K, LB, scale=scale)
    q, k = f32(Q).astype(np.float64), f32(K).astype(np.float64)
    want = np.zeros((3, L))
    for n in range(N):
        P = np.zeros((L, L))
        for i in range(L):
            z = np.array([scale * sum(q[i, n, d] * k[j, n, d] for d in range(D)) for j in range(L)])
            e = np.exp(z - z.max())
            P[i] = e / e.sum()
        for j in range(L):
            lo = lambda i: (i // LB) * LB
            sets = ([i for i in range(L) if j < lo(i)], [i for i in range(L) if lo(i) <= j < lo(i) + LB],
                    [i for i in range(L) if j >= lo(i) + LB])
            for c, I in enumerate(sets):
                want[c, j] += max((P[i, j] for i in I), default=0.0) / N
    assert np.allclose(comp, want, atol=1e-14)
    for j in range(L):
        w = (want[1, j] + want[0, j]) / 2 if j < LB else ((want[2, j] + want[1, j] + want[0, j]) / 3 if j < L - LB
                                                            else (want[1, j] + want[2, j]) / 2)
        assert abs(s[j] - w) < 1e-14


def test_sse_sampled_columns_equal_full_and_dense():
    # the streaming variant used at full size: same numbers as the full oracle, and as dense torch
    rng = np.random.default_rng(8)
    L, N, D, LB = 37, 2, 8, 9
    Q = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    K = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    cols = [0, 8, 9, 17, 18, 27, 28, 35, 36]
    s, comp = oracle.sse(Q, K, LB)
    s2, comp2 = oracle.sse_cols(Q, K, LB, cols)
    assert np.allclose(s2, s[cols], atol=1e-14) and np.allclose(comp2, comp[:, cols], atol=1e-14)
    tq = torch.from_numpy(f32(Q)).double(); tk = torch.from_numpy(f32(K)).double()
    P = torch.softmax(torch.einsum("qnd,knd->nqk", tq, tk) / math.sqrt(D), dim=-1).numpy()
    for ci, j in enumerate(cols):
        qb = np.arange(L) // LB
        for cls, mask in enumerate((qb > j // LB, qb == j // LB, qb < j // LB)):
            want = np.mean([P[n, mask, j].max() if mask.any() else 0.0 for n in range(N)])
            assert abs(comp2[cls, ci] - want) < 1e-13


def test_sse_global_max_against_dense_torch():
    rng = np.random.default_rng(12)
    L, N, D = 19, 3, 8
    Q = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    K = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    g = oracle.sse_global_max(Q, K)
    tq = torch.from_numpy(f32(Q)).double(); tk = torch.from_numpy(f32(K)).double()
    P = torch.softmax(torch.einsum("qnd,knd->nqk", tq, tk) / math.sqrt(D), dim=-1)
    assert np.allclose(g, P.max(dim=1).values.mean(dim=0).numpy(), atol=1e-14)
    a = oracle.sse_global_avg(Q, K)
    assert np.allclose(a, P.mean(dim=1).mean(dim=0).numpy(), atol=1e-14)
    assert abs(a.sum() - 1.0) < 1e-12          # rows of P sum to one, so the column means sum to one
    # it dominates each of the three block-wise components and equals their maximum for one head
    _, comp = oracle.sse(Q[:, :1], K[:, :1], 5)
    assert np.allclose(oracle.sse_global_max(Q[:, :1], K[:, :1]), comp.max(axis=0), atol=1e-14)


def test_sse_mean_first_against_dense_torch_and_index_sets():
    """Algorithm 3's order: the mean over heads comes before the maximum over queries.  Pinned to
    dense torch softmax with the three query classes written as masks, to the explicit index sets
    in Python loops, to the one-head case (where both orders are the same thing) and to the
    inequality max_i mean_n P <= mean_n max_i P."""
    rng = np.random.default_rng(33)
    L, N, D, LB = 23, 3, 8, 6
    Q = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    K = bf(rng.standard_normal((L, N, D)).astype(np.float32) * 2)
    s, comp = oracle.sse_mean_first(Q, K, LB)
    tq = torch.from_numpy(f32(Q)).double(); tk = torch.from_numpy(f32(K)).double()
    A = torch.softmax(torch.einsum("qnd,knd->nqk", tq, tk) / math.sqrt(D), dim=-1).mean(dim=0).numpy()   # [L, L]
    qi = np.arange(L)[:, None]; kj = np.arange(L)[None, :]
    lo = (qi // LB) * LB; hi = lo + LB
    low = np.where(kj < lo, A, 0).max(0); diag = np.where((kj >= lo) & (kj < hi), A, 0).max(0)
    up = np.where(kj >= hi, A, 0).max(0)
    assert np.allclose(comp, np.stack([low, diag, up]), atol=1e-13)
    want = np.where(kj[0] < LB, (diag + low) / 2, np.where(kj[0] < L - LB, (up + diag + low) / 3, (diag + up) / 2))
    assert np.allclose(s, want, atol=1e-13)
    # explicit index sets
    for j in range(L):
        blk = lambda i: i // LB
        sets = ([i for i in range(L) if blk(i) > blk(j)], [i for i in range(L) if blk(i) == blk(j)],
                [i for i in range(L) if blk(i) < blk(j)])
        for c, I in enumerate(sets):
            assert abs(comp[c, j] - max((A[i, j] for i in I), default=0.0)) < 1e-13
    # never above the per-head-maximum-first value of Eq. 4, and different from it for several heads
    s4, comp4 = oracle.sse(Q, K, LB)
    assert np.all(comp <= comp4 + 1e-15) and np.abs(comp - comp4).max() > 1e-3
    # one head: the two orders coincide
    s1, c1 = oracle.sse_mean_first(Q[:, :1], K[:, :1], LB)
    s1b, c1b = oracle.sse(Q[:, :1], K[:, :1], LB)
    assert np.allclose(c1, c1b, atol=1e-15) and np.allclose(s1, s1b, atol=1e-15)
    # uniform attention (zero queries): every class that has queries gives 1 / L
    _, cu = oracle.sse_mean_first(np.zeros_like(Q), K, LB)
    assert np.allclose(cu[1], 1.0 / L, atol=1e-15)


def test_cache_update_is_algorithm2_by_brute_force():
    """Algorithm 2's cache update against a brute-force statement of it: while the chunk fits
    nothing moves; otherwise the survivors are the sink prefix plus the best of the rest by
    (score descending, index ascending), in their old order, the same rows in every layer."""
    rng = np.random.default_rng(5)
    cap, C, n_sink, n_layers = 40, 12, 5, 3
    K = [np.zeros((0, 4), np.uint16) for _ in range(n_layers)]; V = [k.copy() for k in K]
    SL = np.zeros(0, np.float32)
    tags = np.zeros(0, np.int64)                         # global token number of every cached row
    next_tag, pruned = 0, 0
    for c in range(9):
        newK = [rng.integers(0, 65536, (C, 4)).astype(np.uint16) for _ in range(n_layers)]
        newV = [rng.integers(0, 65536, (C, 4)).astype(np.uint16) for _ in range(n_layers)]
        for l in range(n_layers):
            newK[l][:, 0] = np.arange(next_tag, next_tag + C) & 0xffff     # row identity travels with the row
        s_new = rng.integers(0, 6, C).astype(np.float32)                   # many ties
        T = SL.shape[0]
        K2, V2, SL2, ids = oracle.cache_update(K, V, SL, newK, newV, s_new, cap, n_sink)
        if T + C <= cap:
            assert ids is None
            keep = np.arange(T)
        else:
            pruned += 1
            k = cap - C
            rest = sorted(range(n_sink, T), key=lambda i: (-SL[i], i))[: k - n_sink]
            keep = np.array(sorted(list(range(n_sink)) + rest))
            assert np.array_equal(ids, keep) and len(keep) == k
        assert SL2.shape[0] == len(keep) + C <= cap
        assert np.array_equal(SL2, np.concatenate([SL[keep], s_new]))
        for l in range(n_layers):
            assert np.array_equal(K2[l], np.concatenate([K[l][keep], newK[l]]))
            assert np.array_equal(V2[l], np.concatenate([V[l][keep], newV[l]]))
        tags = np.concatenate([tags[keep], np.arange(next_tag, next_tag + C)])
        assert np.array_equal(K2[0][:, 0], tags & 0xffff)
        assert np.array_equal(tags[:n_sink], np.arange(n_sink))            # the sink prefix never leaves
        assert np.all(np.diff(tags) > 0)                                   # temporal order is kept
        K, V, SL, next_tag = K2, V2, SL2, next_tag + C
    assert pruned >= 5
    with pytest.raises(ValueError):
        oracle.cache_update(K, V, SL, [np.zeros((cap + 1, 4), np.uint16)] * n_layers,
                            [np.zeros((cap + 1, 4), np.uint16)] * n_layers, np.zeros(cap + 1, np.float32), cap, n_sink)
