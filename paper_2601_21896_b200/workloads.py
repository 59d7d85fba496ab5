"""Seeded synthetic inputs for the PaFu-KV inference hot path.

This module only *draws inputs*: shapes, random values and their rounding to
bf16 bit patterns.  It holds none of the method's arithmetic (no salience
head, no selection rule, no attention), so the CPU oracle's tests and the CUDA
path's tests can both take their inputs from here without sharing any of the
computation under test.

Every tensor is returned as a numpy ``uint16`` array of bf16 bit patterns
(round-to-nearest-even from fp32), token-major ``[tokens, n_heads, d_head]``,
or as fp32/int64 where noted.  Random numbers come from numpy's counter-based
Philox generator keyed by ``(seed, workload, layer, stream, tensor)``.

Shapes follow the paper's Wan2.1 geometry: 1560 latent tokens per frame
(832x480 video, 8x VAE, 2x2 patches), chunks of 3 frames = 4680 tokens,
12 heads x 128 dims for the 1.3B backbone (Appendix A, "KV Cache and Salience
Score List" and "S-MLP"; Sec. 4.3 "reduced KV Cache size").
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Sequence, Tuple

import numpy as np

TOKENS_PER_FRAME = 1560          # Sec. 4.3: one latent frame = 1560 tokens
CHUNK_TOKENS = 3 * TOKENS_PER_FRAME   # Appendix A: a chunk is 4680 tokens

ACT_GELU = 0   # exact erf form x * Phi(x)
ACT_SILU = 1   # the paper's S-MLP activation (Appendix A, "S-MLP")
FINAL_NONE = 0
FINAL_SIGMOID = 1

_TENSOR_IDS = {"Q": 1, "K": 2, "V": 3, "Kq": 4, "Vq": 5, "w1": 6, "b1": 7, "w2": 8, "b2": 9,
               "UK": 10, "UV": 11, "cK": 12, "cV": 13, "SL": 14, "misc": 15}


@dataclass(frozen=True)
class Workload:
    """One layer's worth of shapes for the hot path (possibly several ragged streams)."""
    name: str
    wid: int                      # key for the random sub-streams
    n_heads: int
    d_head: int
    T: Tuple[int, ...]            # cache length per stream (before pruning)
    budget: Tuple[int, ...]       # retained tokens per stream
    n_sink: int
    n_recent: int
    Lq: Tuple[int, ...]           # chunk query tokens per stream
    d_hidden: int
    d_out: int = 1
    act: int = ACT_GELU
    final: int = FINAL_NONE
    tokens_per_frame: int = TOKENS_PER_FRAME
    structure: str = "iid"        # "iid" | "lowrank" | "lowrank_ar1"
    rank: int = 16
    shared_std: float = 0.5
    rho: float = 0.95
    n_layers: int = 1

    @property
    def d_model(self) -> int:
        return self.n_heads * self.d_head

    @property
    def n_streams(self) -> int:
        return len(self.T)

    def cu(self, what: str) -> np.ndarray:
        vals = {"T": self.T, "B": tuple(min(b, t) for b, t in zip(self.budget, self.T)),
                "Lq": self.Lq}[what]
        return np.concatenate([[0], np.cumsum(vals)]).astype(np.int64)

    def attn_flops(self) -> int:
        """4 * Lq * Lk * D * N summed over streams, Lk = retained + chunk."""
        tot = 0
        for t, b, lq in zip(self.T, self.budget, self.Lq):
            tot += 4 * lq * (min(b, t) + lq) * self.d_head * self.n_heads
        return tot


def tiny() -> Workload:
    return Workload("tiny", 0, n_heads=2, d_head=64, T=(512,), budget=(128,), n_sink=4,
                    n_recent=64, Lq=(64,), d_hidden=32, final=FINAL_SIGMOID,
                    tokens_per_frame=64, structure="iid")


def wan13b_layer(budget_frac: float = 0.5) -> Workload:
    T = 18 * TOKENS_PER_FRAME
    return Workload("wan1.3b_layer", 1, n_heads=12, d_head=128, T=(T,),
                    budget=(int(np.floor(budget_frac * T + 1e-9)),), n_sink=TOKENS_PER_FRAME,
                    n_recent=CHUNK_TOKENS, Lq=(CHUNK_TOKENS,), d_hidden=256,
                    structure="lowrank")


def wan13b_30layer(budget_frac: float = 0.5) -> Workload:
    w = wan13b_layer(budget_frac)
    return replace(w, name="wan1.3b_30layer_b%d" % round(100 * budget_frac), wid=2, n_layers=30)


def long_horizon() -> Workload:
    return Workload("long_horizon", 3, n_heads=12, d_head=128, T=(60 * TOKENS_PER_FRAME,),
                    budget=(9360,), n_sink=TOKENS_PER_FRAME, n_recent=CHUNK_TOKENS,
                    Lq=(CHUNK_TOKENS,), d_hidden=256, structure="lowrank_ar1")


def batch4_14b() -> Workload:
    T = (9360, 18720, 28080, 46800)
    return Workload("batch4_14b", 4, n_heads=40, d_head=128, T=T,
                    budget=tuple(int(np.floor(0.35 * t + 1e-9)) for t in T),
                    n_sink=TOKENS_PER_FRAME, n_recent=TOKENS_PER_FRAME,
                    Lq=(CHUNK_TOKENS,) * 4, d_hidden=512, structure="lowrank")


def paper_native() -> Workload:
    """The paper's own operating point: 4680 history + 4680 new tokens pruned to 4680
    (Sec. 3.4 inference paragraph; Appendix A cache size), no forced recent window."""
    return Workload("paper_native", 5, n_heads=12, d_head=128, T=(2 * CHUNK_TOKENS,),
                    budget=(CHUNK_TOKENS,), n_sink=TOKENS_PER_FRAME, n_recent=0,
                    Lq=(CHUNK_TOKENS,), d_hidden=256, structure="lowrank")


def small_ragged(n_heads: int = 2, d_head: int = 128) -> Workload:
    """A few-tile, ragged-tail, multi-stream case the oracle finishes in seconds."""
    return Workload("small_ragged", 6, n_heads=n_heads, d_head=d_head, T=(700, 333, 1200),
                    budget=(300, 333, 517), n_sink=24, n_recent=72, Lq=(200, 72, 331),
                    d_hidden=64, tokens_per_frame=24, structure="lowrank", rank=4)


CONFIGS = {
    "tiny": tiny, "wan1.3b_layer": wan13b_layer, "wan1.3b_30layer": wan13b_30layer,
    "long_horizon": long_horizon, "batch4_14b": batch4_14b, "paper_native": paper_native,
    "small_ragged": small_ragged,
}


# --------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even); returns uint16 bit patterns. NaN stays NaN."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def rng_for(seed: int, wid: int, layer: int, stream: int, tensor: str) -> np.random.Generator:
    ss = np.random.SeedSequence([int(seed), int(wid), int(layer), int(stream), _TENSOR_IDS[tensor]])
    return np.random.Generator(np.random.Philox(ss))


def _normal(rng: np.random.Generator, shape) -> np.ndarray:
    return rng.standard_normal(shape, dtype=np.float32)


def _tokens_with_frame_structure(w: Workload, seed: int, layer: int, stream: int, tensor: str,
                                 n_tokens: int, first_frame: int,
                                 basis_tensor: str, coef_tensor: str) -> np.ndarray:
    """x_t = eps_t + shared_std * (c_t U_f) / sqrt(rank), U_f a per-frame [rank, d_model] basis.

    "lowrank": U_f i.i.d. per frame.  "lowrank_ar1": U_f = rho U_{f-1} + sqrt(1-rho^2) Xi_f.
    The basis of frame f is the same for cache and chunk tokens of that frame index.
    """
    dm = w.d_model
    x = _normal(rng_for(seed, w.wid, layer, stream, tensor), (n_tokens, dm))
    if w.structure == "iid" or n_tokens == 0:
        return x
    tpf = w.tokens_per_frame
    n_frames = (n_tokens + tpf - 1) // tpf
    last_frame = first_frame + n_frames
    rb = rng_for(seed, w.wid, layer, stream, basis_tensor)
    coef = _normal(rng_for(seed, w.wid, layer, stream, coef_tensor), (n_tokens, w.rank))
    scale = np.float32(w.shared_std / np.sqrt(w.rank))
    U = None
    a = np.float32(w.rho)
    bcoef = np.float32(np.sqrt(1.0 - w.rho * w.rho))
    for f in range(last_frame):
        xi = _normal(rb, (w.rank, dm))
        if w.structure == "lowrank_ar1" and U is not None:
            U = a * U + bcoef * xi
        else:
            U = xi
        if f < first_frame:
            continue
        lo = (f - first_frame) * tpf
        hi = min(lo + tpf, n_tokens)
        x[lo:hi] += scale * (coef[lo:hi] @ U)
    return x


def make_layer(w: Workload, seed: int = 0, layer: int = 0,
               tensors: Sequence[str] = ("Q", "K", "V", "Kq", "Vq", "head")) -> Dict[str, np.ndarray]:
    """Draw one layer's inputs.  Token tensors are packed over streams (stream s owns
    rows [cu[s], cu[s+1])) and shaped [tokens, n_heads, d_head] as uint16 bf16 bits.
    The salience head is ``w1 [d_hidden, d_model]``, ``b1 [d_hidden]``, ``w2 [d_out, d_hidden]``,
    ``b2 [d_out]`` (torch.nn.Linear layout), drawn N(0,1)/sqrt(fan_in)."""
    out: Dict[str, np.ndarray] = {}
    N, D, dm = w.n_heads, w.d_head, w.d_model
    for name in tensors:
        if name == "head":
            out["w1"] = f32_to_bf16_bits(_normal(rng_for(seed, w.wid, layer, 0, "w1"),
                                                  (w.d_hidden, dm)) / np.float32(np.sqrt(dm)))
            out["b1"] = f32_to_bf16_bits(_normal(rng_for(seed, w.wid, layer, 0, "b1"),
                                                  (w.d_hidden,)) / np.float32(np.sqrt(dm)))
            out["w2"] = f32_to_bf16_bits(_normal(rng_for(seed, w.wid, layer, 0, "w2"),
                                                  (w.d_out, w.d_hidden)) / np.float32(np.sqrt(w.d_hidden)))
            out["b2"] = f32_to_bf16_bits(_normal(rng_for(seed, w.wid, layer, 0, "b2"),
                                                  (w.d_out,)) / np.float32(np.sqrt(w.d_hidden)))
            continue
        parts: List[np.ndarray] = []
        for s in range(w.n_streams):
            if name == "Q":
                x = _normal(rng_for(seed, w.wid, layer, s, "Q"), (w.Lq[s], dm))
            elif name in ("K", "V"):
                x = _tokens_with_frame_structure(w, seed, layer, s, name, w.T[s], 0,
                                                 "U" + name, "c" + name)
            elif name in ("Kq", "Vq"):
                first = (w.T[s] + w.tokens_per_frame - 1) // w.tokens_per_frame
                x = _tokens_with_frame_structure(w, seed, layer, s, name, w.Lq[s], first,
                                                 "U" + name[0], "c" + name[0])
            else:
                raise KeyError(name)
            parts.append(f32_to_bf16_bits(x))
        out[name] = np.concatenate(parts, axis=0).reshape(-1, N, D)
    return out


def random_scores(n: int, seed: int = 0, kind: str = "normal", tag: int = 0) -> np.ndarray:
    """fp32 score arrays for selection tests: "normal", "ties" (few distinct values),
    "equal" (all the same), "saturated" (many exact 0/1 as a sigmoid would give),
    "heavy" (heavy-tailed), "signed_zero" (+0/-0 mix)."""
    rng = rng_for(seed, 99, tag, 0, "misc")
    if kind == "normal":
        return rng.standard_normal(n, dtype=np.float32)
    if kind == "ties":
        return rng.integers(0, 4, size=n).astype(np.float32) * np.float32(0.25)
    if kind == "equal":
        return np.full(n, 0.5, dtype=np.float32)
    if kind == "saturated":
        x = rng.standard_normal(n, dtype=np.float32) * np.float32(40.0)
        return (1.0 / (1.0 + np.exp(-x.astype(np.float64)))).astype(np.float32)
    if kind == "heavy":
        return rng.standard_cauchy(n).astype(np.float32)
    if kind == "signed_zero":
        x = np.zeros(n, dtype=np.float32)
        x[rng.integers(0, 2, size=n) == 1] = np.float32(-0.0)
        x[rng.integers(0, 3, size=n) == 0] = rng.standard_normal(1, dtype=np.float32)[0]
        return x
    raise KeyError(kind)


def sample_rows(n_rows: int, n_sample: int, seed: int = 0, tile: int = 128, tag: int = 0) -> np.ndarray:
    """A sorted sample of query rows that always contains the first row, the last row and
    every row of the (possibly partial) last tile boundary region."""
    if n_rows <= n_sample:
        return np.arange(n_rows, dtype=np.int64)
    rng = rng_for(seed, 98, tag, 0, "misc")
    must = {0, n_rows - 1, (n_rows // tile) * tile - 1, min((n_rows // tile) * tile, n_rows - 1)}
    must = {m for m in must if 0 <= m < n_rows}
    rest = rng.choice(n_rows, size=n_sample, replace=False)
    rows = np.array(sorted(must | set(int(r) for r in rest[: n_sample - len(must)])), dtype=np.int64)
    return rows


def peaked_attention_inputs(kind: str, n_heads: int, d_head: int, Lq: int, nB: int, seed: int = 0,
                            q_scale: float = 1.0, rise_per_tile: float = 0.0, spike_pos: Sequence[int] = (),
                            spike_gain: float = 4.0, varied_rows: bool = False, tile: int = 64,
                            tiny_every: int = 3, tiny_gain: float = 5.0) -> Dict[str, np.ndarray]:
    """Inputs whose attention rows are NOT near-uniform (real attention maps are peaked: Sec. 3.2),
    so that a tiled softmax has to move its running maximum.  Returns bf16 bit patterns
    Q [Lq, N, D], Kc/Vc [nB, N, D] (retained segment), Kq/Vq [Lq, N, D] (chunk segment); keys are
    numbered retained first, then chunk.  Every query carries a component g_i along the all-ones
    direction e and key j a component a_j, so logit(i, j) ~ a_j (g_i sqrt(D) + xi_i) + N(0, ~1):

      "scaled_q"    plain Gaussian Q, K with Q multiplied by q_scale (logit spread q_scale nats)
      "ramp"        a_j rises linearly along the key axis by rise_per_tile nats per 64 keys
                    (negative: falls), so the row maximum moves in every tile (or never)
      "spike"       keys at positions spike_pos are spike_gain * e: each dominates its row by
                    ~spike_gain * sqrt(D) nats; the k-th listed spike is (1 + k/2) times stronger,
                    so later ones overtake earlier ones
      "tiny_tiles"  every tiny_every-th 64-key tile of each segment is pushed ~tiny_gain * sqrt(D)
                    nats below the rest: a run that opens on such a tile starts from a far too
                    small maximum
    varied_rows draws g_i uniformly from [-1, 2] instead of 1: in one 32-row group some rows
    see the spike as dominant, some as negligible, some not at all.
    """
    N, D = n_heads, d_head
    rq = rng_for(seed, 97, 0, 0, "Q"); rk = rng_for(seed, 97, 0, 0, "K"); rv = rng_for(seed, 97, 0, 0, "V")
    Q = _normal(rq, (Lq, N, D)); K = _normal(rk, (nB + Lq, N, D)); V = _normal(rv, (nB + Lq, N, D))
    root = np.float32(np.sqrt(D))
    if kind == "scaled_q":
        Q *= np.float32(q_scale)
    else:
        g = np.ones((Lq, 1, 1), np.float32)
        if varied_rows:
            g = rng_for(seed, 97, 0, 0, "misc").uniform(-1.0, 2.0, size=(Lq, 1, 1)).astype(np.float32)
        Q += g
        if kind == "ramp":
            j = np.arange(nB + Lq, dtype=np.float32).reshape(-1, 1, 1)
            K += np.float32(rise_per_tile) * (j / np.float32(tile)) / root
        elif kind == "spike":
            for k, pos in enumerate(spike_pos):
                K[pos] = np.float32(spike_gain * (1.0 + 0.5 * k))
        elif kind == "tiny_tiles":
            for lo, hi in ((0, nB), (nB, nB + Lq)):
                for t0 in range(lo, hi, tile * tiny_every):
                    K[t0:min(t0 + tile, hi)] -= np.float32(tiny_gain)
        else:
            raise KeyError(kind)
    b = f32_to_bf16_bits
    return {"Q": b(Q), "Kc": b(K[:nB]), "Vc": b(V[:nB]), "Kq": b(K[nB:]), "Vq": b(V[nB:])}


def queries_from_keys(w: Workload, d: Dict[str, np.ndarray], seed: int = 0) -> np.ndarray:
    """Replacement for d["Q"]: query i of a stream is a copy (all heads) of one key row the
    retention rule always keeps - a sink or recent row of the cache - or of one of the chunk's own
    key rows, alternating.  q = k makes that key's logit |k|^2 / sqrt(D) ~ 14 nats at these
    input statistics against ~1.3 nats of spread for the others: peaked attention rows."""
    cuT, cuQ = w.cu("T"), w.cu("Lq")
    out = d["Q"].copy()
    for s in range(w.n_streams):
        rng = rng_for(seed, 96, 0, s, "Q")
        T, Lq, B = w.T[s], w.Lq[s], min(w.budget[s], w.T[s])
        nr = min(w.n_recent, B); ns = min(w.n_sink, B - nr)
        always = np.concatenate([np.arange(ns), np.arange(T - nr, T)]) if T > B else np.arange(T)
        for i in range(Lq):
            if (i & 1) and len(always):
                out[cuQ[s] + i] = d["K"][cuT[s] + always[rng.integers(len(always))]]
            else:
                out[cuQ[s] + i] = d["Kq"][cuQ[s] + rng.integers(Lq)]
    return out


def make_layer_device(w: Workload, seed: int = 0, layer: int = 0, device: str = "cuda"):
    """The recipe of make_layer drawn on a CUDA device with torch's counter-based generator: the
    same shapes, law and frame structure, a different random stream (the host version takes
    seconds per layer at full size, which a 30-layer benchmark cannot afford).  Returns torch
    bf16 tensors Q, K, V, Kq, Vq [tokens, n_heads, d_head] and w1, b1, w2, b2."""
    import torch

    N, D, dm = w.n_heads, w.d_head, w.d_model
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(w.wid) * 1009 + int(layer)) & 0x7FFFFFFF)
    rn = lambda *shape: torch.randn(*shape, generator=g, device=device, dtype=torch.float32)

    def tokens(n_tokens: int, first_frame: int, bases):
        x = rn(n_tokens, dm)
        if w.structure == "iid" or n_tokens == 0:
            return x
        tpf = w.tokens_per_frame
        n_frames = (n_tokens + tpf - 1) // tpf
        U = bases(first_frame + n_frames)[first_frame:]                    # [n_frames, rank, dm]
        coef = rn(n_frames * tpf, w.rank).view(n_frames, tpf, w.rank)
        shared = torch.bmm(coef, U).view(n_frames * tpf, dm)[:n_tokens]
        return x + (w.shared_std / float(np.sqrt(w.rank))) * shared

    out = {}
    parts = {k: [] for k in ("Q", "K", "V", "Kq", "Vq")}
    for s in range(w.n_streams):
        first = (w.T[s] + w.tokens_per_frame - 1) // w.tokens_per_frame
        n_total = first + (w.Lq[s] + w.tokens_per_frame - 1) // w.tokens_per_frame
        cache = {}

        def make_bases(tag):
            def bases(n):
                if tag not in cache:
                    xi = rn(n_total, w.rank, dm)
                    if w.structure == "lowrank_ar1":
                        a, b = w.rho, float(np.sqrt(1.0 - w.rho * w.rho))
                        for f in range(1, n_total):
                            xi[f] = a * xi[f - 1] + b * xi[f]
                    cache[tag] = xi
                return cache[tag][:n]
            return bases
        bk, bv = make_bases("K"), make_bases("V")
        parts["Q"].append(rn(w.Lq[s], dm))
        parts["K"].append(tokens(w.T[s], 0, bk)); parts["V"].append(tokens(w.T[s], 0, bv))
        parts["Kq"].append(tokens(w.Lq[s], first, bk)); parts["Vq"].append(tokens(w.Lq[s], first, bv))
        del cache
    for k, v in parts.items():
        out[k] = torch.cat(v, dim=0).to(torch.bfloat16).view(-1, N, D).contiguous()
    out["w1"] = (rn(w.d_hidden, dm) / float(np.sqrt(dm))).to(torch.bfloat16)
    out["b1"] = (rn(w.d_hidden) / float(np.sqrt(dm))).to(torch.bfloat16)
    out["w2"] = (rn(w.d_out, w.d_hidden) / float(np.sqrt(w.d_hidden))).to(torch.bfloat16)
    out["b2"] = (rn(w.d_out) / float(np.sqrt(w.d_hidden))).to(torch.bfloat16)
    return out
