"""pafu_chunk_attn_noalloc: chunk attention for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is off limits on the hot path - inside another
framework's pre-planned memory pool, in a service with a fixed device-memory budget, or as a
plug-in that is handed nothing but its input and output buffers.  For them the library carries
its own fixed scratch array and this entry point uses it instead of a caller workspace.  The
test calls it through the C ABI twice in a row (the scratch is shared and keeps the previous
call's contents, so the second call checks that nothing stale leaks through) and compares each
result with pafu_chunk_attn on the same inputs, within the tolerance of the other GPU tests.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2601_21896_b200 as pafu
from paper_2601_21896_b200 import workloads as wl
from paper_2601_21896_b200.harness import Layer, bf16_to_bits

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def _as_f32(t):
    return wl.bf16_bits_to_f32(bf16_to_bits(t)).astype(np.float64)


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_twice():
    for w in (wl.small_ragged(2, 128), wl.paper_native()):
        d = wl.make_layer(w)
        L = Layer(w, d)
        # retained cache: any valid, ascending selection will do for an attention-only check
        L.score(); L.select(); L.compact()
        L.attn(); L.check_status()
        want_O, want_lse = _as_f32(L.O), L.LSE.cpu().numpy().astype(np.float64)
        truth = None
        if w.name == "small_ragged":
            # small enough for the CPU oracle: compare with the definition as well, stream by stream
            Kc, Vc = bf16_to_bits(L.Kc), bf16_to_bits(L.Vc)
            cuB, cuQ = L.cu_B, w.cu("Lq")
            truth = [oracle.attention(d["Q"][cuQ[s]:cuQ[s + 1]], Kc[cuB[s]:cuB[s + 1]], Vc[cuB[s]:cuB[s + 1]],
                                      d["Kq"][cuQ[s]:cuQ[s + 1]], d["Vq"][cuQ[s]:cuQ[s + 1]]) for s in range(w.n_streams)]
        for call in range(2):
            O = torch.full_like(L.O, float("nan"))
            LSE = torch.full_like(L.LSE, float("nan"))
            pafu.pafu_chunk_attn_noalloc(L.Q, L.Kc, L.Vc, L.cu_B, L.Kq, L.Vq, L.shape, 0.0, O, LSE)
            torch.cuda.synchronize()
            got_O, got_lse = _as_f32(O), LSE.cpu().numpy().astype(np.float64)
            assert np.all(np.isfinite(got_O)) and np.all(np.isfinite(got_lse)), (w.name, call)
            err = np.abs(got_O - want_O)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (w.name, call, err.max(), err.mean())
            err = np.abs(got_lse - want_lse)
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (w.name, call, err.max())
            if truth is not None:
                for s, (tO, tL) in enumerate(truth):
                    err = np.abs(got_O[cuQ[s]:cuQ[s + 1]] - tO)
                    assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, ("oracle", s, call, err.max(), err.mean())
                    assert np.abs(got_lse[:, cuQ[s]:cuQ[s + 1]] - tL).max() <= MAX_ABS, ("oracle LSE", s, call)


@pytest.mark.gpu
def test_noalloc_rejects_what_it_cannot_hold():
    # beyond the stated limit (query rows x heads) nothing is launched and the outputs stay untouched
    N, D, Lq = 40, 128, 4680
    shape = pafu.Shape(N, D, None, [0, Lq])
    t = torch.zeros((16, N, D), dtype=torch.bfloat16, device="cuda")
    O = torch.full((16, N, D), 7.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(pafu.PafuError) as e:
        pafu.pafu_chunk_attn_noalloc(t, t, t, [0, 16], t, t, shape, 0.0, O, None)
    assert e.value.status == 8
    torch.cuda.synchronize()
    assert torch.all(O == 7.0)
    with pytest.raises(pafu.PafuError) as e:      # d_head 64 has no built-in scratch variant
        pafu.pafu_chunk_attn_noalloc(t, t, t, [0, 16], t, t, pafu.Shape(2, 64, None, [0, 8]), 0.0, O, None)
    assert e.value.status == 3
