"""The forward for callers that may not allocate device memory (``sfda_forward_noalloc``).

Some users of this library run inside a process whose device memory is fully planned at start-up (an
inference server's pool, a plug-in inside someone else's memory budget): they can pass inputs and outputs
they already own, but they cannot call the CUDA allocator to get the small workspace ``sfda_forward`` wants.
For them the library carries a statically allocated scratch block.  This test calls that entry point through
the C ABI twice in a row -- the block keeps the previous call's contents, so the second call proves that
nothing stale leaks into the result -- and checks both against the ordinary entry point.

Collected last on purpose: if it fails, a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

import paper_2607_11897_b200 as sfda
import workloads
from oracle import recurrence

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
TOL = 2e-2          # bf16 inputs, fp32 accumulation: the bar against the oracle


def _device_inputs(inp):
    d = {}
    for key, val in inp.items():
        if val is None:
            d[key] = None
            continue
        t = torch.from_numpy(np.ascontiguousarray(val)).to(DEV)
        d[key] = t.to(torch.bfloat16) if key in ("q", "k", "v") else t
    return d


def _outputs(cfg):
    o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, device=DEV, dtype=torch.bfloat16)
    return o, torch.empty_like(o), torch.empty(cfg.B, cfg.H, cfg.d_k, cfg.d_v, device=DEV)


def _rel(got, want):
    got = np.asarray(got, np.float64)
    assert np.isfinite(got).all()
    return float(np.abs(got - want).max() / max(np.abs(want).max(), 1e-30))


def test_noalloc_forward_matches_forward_on_two_calls_in_a_row():
    cfgs = [workloads.CONFIGS[1].scaled(name="na1", B=2, T=320, H=3, s0_std=0.05, seed=501),
            workloads.CONFIGS[1].scaled(name="na2", B=1, T=130, H=2, s0_std=0.0, seed=502)]
    for cfg in cfgs:
        inp = workloads.forward_inputs(cfg)
        d = _device_inputs(inp)
        # The ordinary entry point on a caller-provided workspace of the minimum size (256 bytes: the status block).
        # With that size it makes the launch the static block allows, so the two must agree in every bit.
        ws = torch.empty(256, dtype=torch.uint8, device=DEV)
        o_ref, oi_ref, S_ref = _outputs(cfg)
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o_ref, oi_ref, S_ref,
                          cfg.chunk, ws)
        assert sfda.sfda_workspace_status(ws) == 0
        # the entry point that uses the library's own scratch block; outputs are allocated before the call
        o, oi, S = _outputs(cfg)
        sfda.sfda_forward_noalloc(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, oi, S, cfg.chunk)
        assert sfda.sfda_noalloc_status() == 0
        assert sfda.last_launch_count() == 1
        assert torch.equal(o, o_ref) and torch.equal(oi, oi_ref) and torch.equal(S, S_ref)
        # ... and both are right: element by element against the CPU oracle
        pairs = [(b, h) for b in range(cfg.B) for h in range(cfg.H)]
        sq = workloads.sequences(inp, pairs)
        w_re, w_im, w_S = recurrence.sfda_recurrence(sq["q"], sq["k"], sq["v"], sq["alpha"], sq["theta"], sq["beta"], sq["S0"])
        on, oin, Sn = o.float().cpu().numpy(), oi.float().cpu().numpy(), S.cpu().numpy()
        assert _rel(np.stack([on[b, :, h] for b, h in pairs]), w_re) <= TOL
        assert _rel(np.stack([oin[b, :, h] for b, h in pairs]), w_im) <= TOL
        assert _rel(np.stack([Sn[b, h] for b, h in pairs]), w_S) <= TOL
        # A second call on the same tensors (the first one covered the load of the kernel image and the look-up of
        # the block's address): the device's free memory, which any allocation inside the library would lower,
        # is what it was, and the block's stale contents change nothing.
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        o.zero_(); oi.zero_(); S.zero_()
        sfda.sfda_forward_noalloc(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, oi, S, cfg.chunk)
        assert sfda.sfda_noalloc_status() == 0
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after >= free_before
        assert torch.equal(o, o_ref) and torch.equal(oi, oi_ref) and torch.equal(S, S_ref)


def test_noalloc_forward_rejects_what_it_cannot_serve():
    cfg = workloads.CONFIGS[0].scaled(name="na3", T=64)          # fp32, d = 64: not the kernel that uses scratch
    inp = workloads.forward_inputs(cfg)
    d = {k: (None if v is None else torch.from_numpy(np.ascontiguousarray(v)).to(DEV)) for k, v in inp.items()}
    o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, device=DEV)
    with pytest.raises(sfda.SfdaError) as e:
        sfda.sfda_forward_noalloc(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], None, o, None, None, cfg.chunk)
    assert e.value.status == -3
