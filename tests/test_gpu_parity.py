"""GPU parity: every entry point of the C-ABI library against the CPU oracle,
element by element, on the same seeded inputs.

Error measure (the paper defines none): err = max|x - y| / max|y| per output
tensor, with y the oracle.  Bars: 1e-4 for fp32 inputs, 2e-2 for bf16 inputs with
fp32 accumulation; integer bookkeeping (chunk plan, cumulative phase turns) must be
bit-exact.
"""
import numpy as np
import pytest
import torch

import paper_2607_11897_b200 as sfda
import workloads
from oracle import backward, bookkeeping, chunk_wy, frontend, recurrence

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-4, "bf16": 2e-2}
DEV = "cuda:0"


def rel_err(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert np.isfinite(got).all(), "non-finite GPU output"
    return float(np.abs(got - want).max() / max(np.abs(want).max(), 1e-30))


def to_dev(x, cfg, key):
    t = torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
    if key in ("q", "k", "v") and cfg.dtype == "bf16":
        t = t.to(torch.bfloat16)          # exact: the values already lie on the bf16 grid
    return t


def run_forward(cfg, inp, want_im=True, simt=False, want_state=True):
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    B, T, H = d["q"].shape[:3]
    o = torch.empty(B, T, H, cfg.d_v, device=DEV, dtype=d["q"].dtype)
    o_im = torch.empty_like(o) if want_im else None
    S_T = torch.empty(B, H, cfg.d_k, cfg.d_v, device=DEV, dtype=torch.float32) if want_state else None
    ws_bytes = sfda.sfda_workspace_bytes(B, T, H, cfg.d_k, cfg.d_v, cfg.chunk, 1 if cfg.dtype == "bf16" else 0)
    ws = torch.empty(max(ws_bytes, 16), device=DEV, dtype=torch.uint8)
    if simt:
        sfda.sfda_forward_simt(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T,
                               cfg.chunk)
    else:
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T,
                          cfg.chunk, ws)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() >= 1
    if ws_bytes and not simt:
        assert sfda.sfda_workspace_status(ws) == 0
    return (o.float().cpu().numpy(), None if o_im is None else o_im.float().cpu().numpy(),
            None if S_T is None else S_T.cpu().numpy())


def oracle_pairs(inp, pairs):
    s = workloads.sequences(inp, pairs)
    return recurrence.sfda_recurrence(s["q"], s["k"], s["v"], s["alpha"], s["theta"], s["beta"], s["S0"])


def check_forward(cfg, inp, pairs, tol, **kw):
    o, o_im, S_T = run_forward(cfg, inp, **kw)
    w_re, w_im, w_S = oracle_pairs(inp, pairs)
    g_re = np.stack([o[b, :, h] for b, h in pairs])
    errs = {"o_re": rel_err(g_re, w_re)}
    if o_im is not None:
        errs["o_im"] = rel_err(np.stack([o_im[b, :, h] for b, h in pairs]), w_im)
    if S_T is not None:
        errs["S_T"] = rel_err(np.stack([S_T[b, h] for b, h in pairs]), w_S)
    for name, e in errs.items():
        assert e <= tol, "%s: %s rel err %.3e > %.1e (%s)" % (cfg.name, name, e, tol, errs)
    return errs


def all_pairs(cfg):
    return [(b, h) for b in range(cfg.B) for h in range(cfg.H)]


# Regression guards of the bf16 tensor-core forward, beside the pass / fail bar TOL["bf16"] = 2e-2 of the task: the
# measured errors are 5e-3 to 8e-3 (maximum) and 4.4e-3 to 4.6e-3 (root mean square, relative) on every
# configuration; 1.5 times that must not be passed without somebody looking.
GUARD_MAX, GUARD_RMS = 1.2e-2, 7.0e-3


class ErrAcc:
    """max |x - y| / max |y| and rms(x - y) / rms(y) of one output tensor, accumulated over batches of sequences."""

    def __init__(self):
        self.dmax = self.ymax = self.d2 = self.y2 = 0.0
        self.n = 0

    def add(self, got, want):
        got = np.asarray(got, np.float64)
        assert np.isfinite(got).all(), "non-finite GPU output"
        d = got - want
        self.dmax = max(self.dmax, float(np.abs(d).max()))
        self.ymax = max(self.ymax, float(np.abs(want).max()))
        self.d2 += float((d * d).sum())
        self.y2 += float((want * want).sum())
        self.n += d.size

    @property
    def max_rel(self):
        return self.dmax / max(self.ymax, 1e-30)

    @property
    def rms_rel(self):
        return float(np.sqrt(self.d2 / max(self.y2, 1e-300)))


def check_all_sequences(name, pairs, oracle_batch, outputs, tol, guard=True, batch=64):
    """Every sequence of `pairs` against the oracle, `batch` sequences at a time (what host memory holds);
    `oracle_batch(sub_pairs)` returns the oracle's (o_re, o_im, S_T) of those sequences, `outputs` the GPU's
    (o [B,T,H,dv], o_im or None, S_T [B,H,dk,dv] or None).  Prints and checks both error figures per tensor."""
    o, o_im, S_T = outputs
    acc = {"o_re": ErrAcc(), "o_im": ErrAcc(), "S_T": ErrAcc()}
    for i in range(0, len(pairs), batch):
        sub = pairs[i:i + batch]
        w_re, w_im, w_S = oracle_batch(sub)
        acc["o_re"].add(np.stack([o[b, :, h] for b, h in sub]), w_re)
        if o_im is not None:
            acc["o_im"].add(np.stack([o_im[b, :, h] for b, h in sub]), w_im)
        if S_T is not None:
            acc["S_T"].add(np.stack([S_T[b, h] for b, h in sub]), w_S)
    report = {k: (a.max_rel, a.rms_rel) for k, a in acc.items() if a.n}
    print("%s: %d sequences; max rel / rms rel: %s" % (
        name, len(pairs), ", ".join("%s %.2e / %.2e" % (k, m, r) for k, (m, r) in report.items())))
    for k, (m, r) in report.items():
        assert m <= tol, "%s: %s max rel err %.3e above the bar %.1e" % (name, k, m, tol)
        if guard:
            assert m <= GUARD_MAX, "%s: %s max rel err %.3e above the regression guard %.1e" % (name, k, m, GUARD_MAX)
            assert r <= GUARD_RMS, "%s: %s rms rel err %.3e above the regression guard %.1e" % (name, k, r, GUARD_RMS)
    return report


# ------------------------------------------------------------------------------------------------
# forward
# ------------------------------------------------------------------------------------------------
def test_forward_cfg0_tiny_fp32():
    cfg = workloads.CONFIGS[0]
    inp = workloads.forward_inputs(cfg)
    check_forward(cfg, inp, all_pairs(cfg), TOL["f32"])


@pytest.mark.parametrize("d_k,d_v,chunk,T", [(64, 64, 16, 100), (64, 128, 32, 77), (128, 64, 64, 130),
                                             (128, 128, 64, 200), (128, 128, 32, 64), (128, 128, 16, 33),
                                             (64, 64, 64, 1), (128, 128, 64, 5)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_forward_simt_shapes_ragged_tail_and_state(d_k, d_v, chunk, T, dtype):
    cfg = workloads.CONFIGS[0].scaled(name="t", B=2, T=T, H=3, d_k=d_k, d_v=d_v, chunk=chunk, dtype=dtype,
                                      s0_std=0.5, seed=100 + d_k + d_v + chunk + T)
    inp = workloads.forward_inputs(cfg)
    # the fp32 path with bf16 storage only rounds the stored outputs: 2^-9 relative
    check_forward(cfg, inp, all_pairs(cfg), 1e-4 if dtype == "f32" else 5e-3, simt=True)


@pytest.mark.parametrize("alpha,beta", [("u(0.3,1)", "u(0,1)"), ("u(0.0,1)", "u(0,1)"),
                                        ("u(0.9,1)", "bernoulli(0.05)"), ("u(1.0,1.0)", "u(0,1)")])
def test_forward_simt_decay_and_write_edges(alpha, beta):
    cfg = workloads.CONFIGS[0].scaled(name="edge", B=1, T=192, H=2, d_k=128, d_v=64, chunk=64, alpha=alpha,
                                      beta=beta, s0_std=1.0, seed=7)
    inp = workloads.forward_inputs(cfg)
    if alpha == "u(0.0,1)":
        inp["alpha"][:, ::17, :, ::5] = 0.0            # exact zeros are admissible (alpha in [0, 1])
    check_forward(cfg, inp, all_pairs(cfg), 1e-4, simt=True)


def test_forward_beta_all_zero_and_all_one():
    for val in (0.0, 1.0):
        cfg = workloads.CONFIGS[0].scaled(name="b", B=1, T=96, H=2, chunk=32, s0_std=1.0, seed=9)
        inp = workloads.forward_inputs(cfg)
        inp["beta"][:] = val
        check_forward(cfg, inp, all_pairs(cfg), 1e-4, simt=True)


def test_forward_outputs_optional():
    cfg = workloads.CONFIGS[0].scaled(name="opt", T=64, seed=3)
    inp = workloads.forward_inputs(cfg)
    check_forward(cfg, inp, all_pairs(cfg), 1e-4, want_im=False, want_state=False)


def test_forward_split_sequence_continues_from_state():
    """forward(T1) then forward(T2, S0 = S_T1) equals forward(T1 + T2) (Theorem "Chunk-bounded exactness")."""
    cfg = workloads.CONFIGS[0].scaled(name="split", T=160, seed=4)
    inp = workloads.forward_inputs(cfg)
    o, o_im, S_T = run_forward(cfg, inp)
    T1 = 64
    first = {k: (None if v is None else v[:, :T1]) for k, v in inp.items()}
    o1, _, S1 = run_forward(cfg, first)
    second = {k: (None if v is None else v[:, T1:]) for k, v in inp.items()}
    second["S0"] = S1
    o2, _, S2 = run_forward(cfg, second)
    assert rel_err(np.concatenate([o1, o2], 1), o) < 1e-5
    assert rel_err(S2, S_T) < 1e-5


@pytest.mark.parametrize("T,H,s0,alpha", [(64, 1, 0.0, "sigmoid(n(3,1))"), (256, 2, 0.02, "sigmoid(n(3,1))"),
                                         (200, 3, 0.5, "sigmoid(n(3,1))"), (1, 2, 1.0, "sigmoid(n(3,1))"),
                                         (130, 2, 1.0, "u(0.5,1)"), (192, 2, 0.3, "u(1.0,1.0)"),
                                         (192, 2, 0.3, "u(0.3,1)")])
def test_forward_tensor_core_path(T, H, s0, alpha):
    """bf16, d_k = d_v = 128, chunk = 64: the tcgen05 path, several chunks, ragged tails, nonzero S0."""
    cfg = workloads.CONFIGS[1].scaled(name="tc", B=2, T=T, H=H, s0_std=s0, alpha=alpha, seed=40 + T)
    assert sfda.sfda_workspace_bytes(cfg.B, T, H, 128, 128, 64, 1) > 0          # takes the tensor-core path
    inp = workloads.forward_inputs(cfg)
    errs = check_forward(cfg, inp, all_pairs(cfg), TOL["bf16"])
    print(errs)


def test_forward_tensor_core_time_slices():
    """More sequences than SMs: the launcher cuts every sequence into time slices that hand their boundary
    state over through the workspace; with only the status block as workspace it does not.  Same results."""
    cfg = workloads.CONFIGS[1].scaled(name="slices", B=5, T=512, H=40, s0_std=0.05, seed=91)
    inp = workloads.forward_inputs(cfg)
    pairs = [(0, 0), (4, 39), (2, 17), (3, 5), (1, 30), (4, 0)]
    check_forward(cfg, inp, pairs, TOL["bf16"])
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    outs = []
    for nbytes in (sfda.sfda_workspace_bytes(cfg.B, cfg.T, cfg.H, 128, 128, 64, 1), 256):
        o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.empty_like(o), torch.empty(cfg.B, cfg.H, 128, 128, device=DEV)
        ws = torch.empty(nbytes, device=DEV, dtype=torch.uint8)
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, 64, ws)
        assert sfda.sfda_workspace_status(ws) == 0
        outs.append((o.float().cpu().numpy(), o_im.float().cpu().numpy(), S_T.cpu().numpy()))
    for x, y in zip(*outs):
        assert np.array_equal(x, y)          # slicing only moves the fp32 state through memory: bit-identical


def test_forward_tensor_core_balanced_partition():
    """304 sequences of nine chunks (an odd count, which time slices cannot halve; the last chunk a ragged tail
    of 63 tokens): the launcher cuts the chunks of all sequences, laid end to end, into one contiguous range per
    CTA, so most sequences are cut once, at different places, and continue on a neighbouring CTA through the
    workspace.  Checked against the oracle on sequences cut early, late and not at all, and bit for bit against
    the same call with only the status block as workspace (no cuts)."""
    cfg = workloads.CONFIGS[1].scaled(name="balanced", B=16, T=575, H=19, s0_std=0.05, seed=93)
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    full = sfda.sfda_workspace_bytes(cfg.B, cfg.T, cfg.H, 128, 128, 64, 1)
    assert sfda.sfda_forward_partition(cfg.B, cfg.T, cfg.H, 128, 128, 64, 1, full, n_sm)[:2] == (1, 1)
    assert sfda.sfda_forward_partition(cfg.B, cfg.T, cfg.H, 128, 128, 64, 1, 256, n_sm)[:2] == (1, 0)
    inp = workloads.forward_inputs(cfg)
    pairs = [(0, 0), (0, 1), (0, 2), (7, 9), (8, 0), (15, 17), (15, 18)]
    check_forward(cfg, inp, pairs, TOL["bf16"])
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    outs = []
    for nbytes in (sfda.sfda_workspace_bytes(cfg.B, cfg.T, cfg.H, 128, 128, 64, 1), 256):
        o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.empty_like(o), torch.empty(cfg.B, cfg.H, 128, 128, device=DEV)
        ws = torch.empty(nbytes, device=DEV, dtype=torch.uint8)
        for _ in range(2):          # the second call finds the first call's counters in the workspace
            sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, 64, ws)
            assert sfda.sfda_workspace_status(ws) == 0
        outs.append((o.float().cpu().numpy(), o_im.float().cpu().numpy(), S_T.cpu().numpy()))
    for x, y in zip(*outs):
        assert np.array_equal(x, y)


def _random_tensor_core_shapes():
    """Fourteen seeded shapes around the launcher's decisions: fewer and more (batch, head) pairs than SMs, chunk counts
    that halve and that do not, T below one tile, exact multiples and ragged tails, with and without S0."""
    rng = np.random.default_rng(20260711)
    shapes = [(1, 1, 1, 0.0), (1, 63, 149, 0.1), (3, 64 * 9, 50, 0.0), (2, 64 * 16 + 1, 75, 0.05),
              (4, 64 * 7 + 5, 60, 0.05), (2, 64 * 12, 100, 0.0)]
    while len(shapes) < 14:
        B, H = int(rng.integers(1, 6)), int(rng.integers(1, 80))
        T = int(rng.integers(1, 40)) * 64 + int(rng.integers(0, 64)) * int(rng.integers(0, 2))
        if B * T * H <= 700_000:
            shapes.append((B, T, H, float(rng.choice([0.0, 0.05, 0.5]))))
    return shapes


@pytest.mark.parametrize("B,T,H,s0", _random_tensor_core_shapes())
def test_forward_tensor_core_random_shapes(B, T, H, s0):
    """The tensor-core forward on seeded random shapes: first, last and three random sequences against the oracle at
    the bar and the regression guards, and the whole output bit for bit against the same call with only the status
    block as workspace (the launcher then cuts nothing)."""
    cfg = workloads.CONFIGS[1].scaled(name="rnd_%d_%d_%d" % (B, T, H), B=B, T=T, H=H, s0_std=s0, seed=7000 + B + T + H)
    inp = workloads.forward_inputs(cfg)
    rng = np.random.default_rng(cfg.seed)
    pairs = sorted({(0, 0), (B - 1, H - 1)} | {(int(rng.integers(B)), int(rng.integers(H))) for _ in range(3)})
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    outs = []
    for nbytes in (sfda.sfda_workspace_bytes(B, T, H, 128, 128, 64, 1), 256):
        o = torch.full((B, T, H, 128), float("nan"), device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.full_like(o, float("nan")), torch.full((B, H, 128, 128), float("nan"), device=DEV)
        ws = torch.empty(nbytes, device=DEV, dtype=torch.uint8)
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, 64, ws)
        assert sfda.sfda_workspace_status(ws) == 0 and sfda.last_launch_count() == 1
        outs.append((o.float().cpu().numpy(), o_im.float().cpu().numpy(), S_T.cpu().numpy()))
    for x, y in zip(*outs):
        assert np.isfinite(x).all() and np.array_equal(x, y)
    check_all_sequences(cfg.name, pairs, lambda sub: oracle_pairs(inp, sub), outs[0], TOL["bf16"], guard=T >= 64)


@pytest.mark.parametrize("case", ["product_exactly_e-80", "product_e-77", "product_e-40_uneven"])
def test_forward_tensor_core_at_the_documented_decay_edge(case):
    """The tensor-core path forms 1 / |gamma_t| inside a chunk and documents prod_chunk alpha >= e^-80 per coordinate
    as its precondition.  Parity must hold up to that edge: a constant alpha = e^-1.25 (product over 64 tokens
    e^-80), e^-1.2 (e^-76.8), and an uneven case (a third of the tokens at e^-1.8, the rest near 1)."""
    cfg = workloads.CONFIGS[1].scaled(name="edge_" + case, B=1, T=256, H=3, s0_std=0.5, seed=321)
    inp = dict(workloads.forward_inputs(cfg))
    rng = np.random.default_rng(99)
    if case == "product_exactly_e-80":
        inp["alpha"] = np.full(inp["alpha"].shape, np.exp(-1.25), np.float32)
    elif case == "product_e-77":
        inp["alpha"] = np.full(inp["alpha"].shape, np.exp(-1.2), np.float32)
    else:
        strong = rng.uniform(0, 1, inp["alpha"].shape) < 1.0 / 3.0
        inp["alpha"] = np.where(strong, np.exp(-1.8), rng.uniform(0.98, 1.0, inp["alpha"].shape)).astype(np.float32)
    check_forward(cfg, inp, all_pairs(cfg), TOL["bf16"])


@pytest.mark.parametrize("case", ["some_alpha_zero", "all_alpha_tiny", "alpha_u(0,1)"])
def test_forward_tensor_core_beyond_the_decay_edge_stays_finite(case):
    """Beyond the documented precondition (alpha = 0 is admissible in the recurrence, Section 3; Prop. "Basic
    numerical stability") the tensor-core path promises finite results, not accuracy: every output and the final
    state must be finite numbers, and the status must stay clean."""
    cfg = workloads.CONFIGS[1].scaled(name="beyond_" + case, B=2, T=200, H=2, s0_std=0.5, seed=322)
    inp = dict(workloads.forward_inputs(cfg))
    rng = np.random.default_rng(98)
    if case == "some_alpha_zero":
        a = inp["alpha"].copy()
        a[rng.uniform(0, 1, a.shape) < 0.1] = 0.0
        inp["alpha"] = a
    elif case == "all_alpha_tiny":
        inp["alpha"] = np.full(inp["alpha"].shape, 1e-20, np.float32)
    else:
        inp["alpha"] = rng.uniform(0.0, 1.0, inp["alpha"].shape).astype(np.float32)
    o, o_im, S_T = run_forward(cfg, inp)            # run_forward checks the status word
    assert np.isfinite(o).all() and np.isfinite(o_im).all() and np.isfinite(S_T).all()
    # the same inputs on the fp32 path, which has no such precondition, agree with the oracle
    w = oracle_pairs(inp, all_pairs(cfg))
    a = run_forward(cfg, inp, simt=True)
    assert rel_err(np.stack([a[0][b, :, h] for b, h in all_pairs(cfg)]), w[0]) <= 5e-3


def test_forward_tensor_core_optional_outputs_and_zero_state():
    """Tensor-core path without o_im, without S_T, and with S0 = NULL (zero state)."""
    cfg = workloads.CONFIGS[1].scaled(name="tc_opt", B=1, T=300, H=2, s0_std=0.0, seed=55)
    inp = workloads.forward_inputs(cfg)
    assert inp["S0"] is None or not np.any(inp["S0"])
    inp["S0"] = None
    check_forward(cfg, inp, all_pairs(cfg), TOL["bf16"], want_im=False, want_state=False)
    check_forward(cfg, inp, all_pairs(cfg), TOL["bf16"], want_im=True, want_state=True)


def test_forward_tensor_core_large_phases_and_write_extremes():
    """Phases far outside (-pi, pi] (the kernel's sines and cosines reduce them), beta = 0 and beta = 1 tokens."""
    cfg = workloads.CONFIGS[1].scaled(name="tc_phase", B=1, T=256, H=2, s0_std=0.3, seed=56)
    inp = workloads.forward_inputs(cfg)
    rng = np.random.default_rng(560)
    inp["theta"] = (inp["theta"] + 2.0 * np.pi * rng.integers(-40, 41, inp["theta"].shape)).astype(np.float32)
    inp["beta"][:, ::3] = 0.0
    inp["beta"][:, 1::3] = 1.0
    check_forward(cfg, inp, all_pairs(cfg), TOL["bf16"])


def test_forward_tensor_core_time_slices_with_ragged_tail():
    """Time slices whose last chunk is a ragged tail (T = 500: eight chunks, the last of 52 tokens)."""
    cfg = workloads.CONFIGS[1].scaled(name="slices_tail", B=5, T=500, H=40, s0_std=0.05, seed=92)
    inp = workloads.forward_inputs(cfg)
    check_forward(cfg, inp, [(0, 0), (4, 39), (2, 20), (3, 7)], TOL["bf16"])


def test_forward_tensor_core_is_deterministic():
    """Two launches on the same inputs give bit-identical results (no atomics or order-dependent sums on the path)."""
    cfg = workloads.CONFIGS[1].scaled(name="det", B=3, T=1024, H=60, s0_std=0.05, seed=93)   # 180 sequences: sliced
    inp = workloads.forward_inputs(cfg)
    a = run_forward(cfg, inp)
    b = run_forward(cfg, inp)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_forward_tensor_core_is_deterministic_at_the_headline_sizes():
    """Five launches of the plain and of the fused forward at B = 8, T = 8192, H = 32: every bit of o, o_im and S_T
    the same.  (32768 chunks per launch: enough for a rare ordering hazard between the roles of the kernel to show;
    a product released by the first half of an operand once overwrote accumulator columns whose second half a slow
    warp had not read yet, in about one chunk per million.)"""
    B, T, H, d = 8, 8192, 32, 128
    g = torch.Generator(device=DEV)
    g.manual_seed(94)
    rn = lambda *s: torch.randn(*s, device=DEV, generator=g)
    q, v = rn(B, T, H, d).to(torch.bfloat16), rn(B, T, H, d).to(torch.bfloat16)
    k = rn(B, T, H, d)
    k = (k / k.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
    a = torch.sigmoid(3.0 + rn(B, T, H, d // 2))
    b = (torch.rand(B, T, H, d // 2, device=DEV, generator=g) * 2 - 1) * np.pi
    c, S0 = torch.sigmoid(rn(B, T, H)), 0.02 * rn(B, H, d, d)

    def run(fused):
        o = torch.empty(B, T, H, d, device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.empty_like(o), torch.empty(B, H, d, d, device=DEV)
        if fused:      # the same arrays read as raw inputs of the stable parameterisation
            ws = torch.empty(sfda.sfda_forward_fused_workspace_bytes(B, T, H, d, d, 64, 1), dtype=torch.uint8, device=DEV)
            sfda.sfda_forward_fused(q, k, v, a, b, c, 0.0, 1.0, float(np.pi), 1e-6, S0, o, o_im, S_T, 64, ws)
        else:
            ws = torch.empty(sfda.sfda_workspace_bytes(B, T, H, d, d, 64, 1), dtype=torch.uint8, device=DEV)
            sfda.sfda_forward(q, k, v, a, b, c, S0, o, o_im, S_T, 64, ws)
        torch.cuda.synchronize()
        assert sfda.sfda_workspace_status(ws) == 0
        return o, o_im, S_T

    for fused in (False, True):
        first = run(fused)
        for _ in range(4):
            again = run(fused)
            for x, y in zip(first, again):
                assert torch.equal(x, y), "fused" if fused else "plain"


def test_forward_tensor_core_matches_cuda_core_path():
    cfg = workloads.CONFIGS[1].scaled(name="tc2", B=1, T=512, H=4, s0_std=0.1, seed=77)
    inp = workloads.forward_inputs(cfg)
    a = run_forward(cfg, inp)
    b = run_forward(cfg, inp, simt=True)
    for x, y in zip(a, b):
        assert rel_err(x, y) < TOL["bf16"]


@pytest.mark.parametrize("idx", [1, 2])
def test_forward_full_size_bf16_configs_all_sequences(idx):
    """Configurations 1 and 2 at full size, in the launch configuration bench.py times (configuration 2: 148
    persistent CTAs, every sequence cut into time slices that hand their state over): EVERY (batch, head) sequence
    against the oracle, element by element, so that a fault tied to a CTA, a slice boundary or a hand-off shows."""
    cfg = workloads.CONFIGS[idx]
    inp = workloads.forward_inputs(cfg)
    out = run_forward(cfg, inp)
    check_all_sequences(cfg.name, all_pairs(cfg), lambda sub: oracle_pairs(inp, sub), out, TOL["bf16"])


def test_forward_long_context_stability():
    """Configuration 3 (T = 131072): parity on all 16 sequences, finite outputs, the Frobenius
    bound of Prop. "Basic numerical stability", bit-exact cumulative phase turns."""
    cfg = workloads.CONFIGS[3]
    inp = workloads.forward_inputs(cfg)
    o, o_im, S_T = run_forward(cfg, inp)
    assert np.isfinite(o).all() and np.isfinite(o_im).all() and np.isfinite(S_T).all()
    check_all_sequences(cfg.name, all_pairs(cfg), lambda sub: oracle_pairs(inp, sub), (o, o_im, S_T), TOL["bf16"], batch=8)
    # ||S_T||_F <= ||S_0||_F + sum beta |k| |v|
    for h in range(cfg.H):
        bound = np.sum(inp["beta"][0, :, h].astype(np.float64)
                       * np.linalg.norm(inp["k"][0, :, h].astype(np.float64), axis=-1)
                       * np.linalg.norm(inp["v"][0, :, h].astype(np.float64), axis=-1))
        assert np.linalg.norm(S_T[0, h].astype(np.float64)) <= bound * (1 + 1e-2) + 1e-6
    k = to_dev(inp["k"], cfg, "k")
    turns = torch.empty(cfg.B, cfg.T, cfg.H, cfg.m, device=DEV, dtype=torch.int32)
    sfda.sfda_chunk_factors(k, to_dev(inp["alpha"], cfg, "alpha"), to_dev(inp["theta"], cfg, "theta"),
                            to_dev(inp["beta"], cfg, "beta"), None, None, None, None, turns, cfg.chunk)
    torch.cuda.synchronize()
    got = turns.cpu().numpy().view(np.uint32)
    want = np.moveaxis(bookkeeping.cumulative_phase_turns(np.moveaxis(inp["theta"], 1, 2), cfg.chunk), 2, 1)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------------------------------------
# factor export
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,B,T,H,full_ws", [("cfg1", 2, 4096, 16, True), ("cfg1_ragged", 1, 1029, 3, False),
                                                ("cfg3", 1, 131072, 16, True), ("cfg2_slices", 8, 2048, 32, True)])
def test_tensor_core_forward_phase_bookkeeping_is_bit_exact(name, B, T, H, full_ws):
    """The integer cumulative phase of the tensor-core kernel (what its rotations are derived from), chunk by chunk,
    against the oracle's emulation of the same single-precision conversion: every bit, with the sequences cut into
    time slices (full workspace) and uncut (256-byte workspace), on uniform and on quantised phases."""
    base = workloads.CONFIGS[3] if name == "cfg3" else workloads.CONFIGS[2 if name == "cfg2_slices" else 1]
    cfg = base.scaled(B=B, T=T, H=H)
    inp = workloads.forward_inputs(cfg)
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    NC = (T + 63) // 64
    o = torch.empty(B, T, H, 128, device=DEV, dtype=torch.bfloat16)
    S_T = torch.empty(B, H, 128, 128, device=DEV)
    ph = torch.full((B, H, NC, 64), -1, device=DEV, dtype=torch.int32)
    nws = sfda.sfda_workspace_bytes(B, T, H, 128, 128, 64, 1) if full_ws else 256
    ws = torch.empty(nws, device=DEV, dtype=torch.uint8)
    sfda.sfda_forward_phase(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, None, S_T, ph, 64, ws)
    torch.cuda.synchronize()
    assert sfda.sfda_workspace_status(ws) == 0
    got = ph.cpu().numpy().view(np.uint32)                                   # [B][H][NC][m]
    want = bookkeeping.chunk_closing_turns_f32(np.moveaxis(inp["theta"], 2, 1), 64)   # theta [B][T][H][m] -> [B][H][T][m]
    assert got.shape == want.shape
    assert np.array_equal(got, want)
    # the same launch still computes the forward: same bits as the plain entry point
    o2 = torch.empty_like(o)
    S2 = torch.empty_like(S_T)
    sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o2, None, S2, 64, ws)
    torch.cuda.synchronize()
    assert torch.equal(o, o2) and torch.equal(S_T, S2)


@pytest.mark.parametrize("d_k,chunk,T,dtype", [(64, 16, 50, "f32"), (128, 64, 150, "f32"), (128, 32, 64, "bf16"),
                                               (64, 64, 64, "f32")])
def test_chunk_factors_match_constructive_recursion(d_k, chunk, T, dtype):
    cfg = workloads.CONFIGS[0].scaled(name="fac", B=2, T=T, H=2, d_k=d_k, chunk=chunk, dtype=dtype, seed=5 + T)
    inp = workloads.forward_inputs(cfg)
    B, H, m, C = cfg.B, cfg.H, cfg.m, chunk
    NC, tail = sfda.sfda_plan(T, chunk)
    assert (NC, tail) == bookkeeping.chunk_plan(T, chunk)
    G = torch.full((B, H, NC, m, 2), float("nan"), device=DEV)
    Y = torch.full((B, H, NC, m, C, 2), float("nan"), device=DEV)
    M = torch.full((B, H, NC, C, C, 2), float("nan"), device=DEV)
    W = torch.full((B, H, NC, m, C, 2), float("nan"), device=DEV)
    turns = torch.zeros(B, T, H, m, device=DEV, dtype=torch.int32)
    sfda.sfda_chunk_factors(to_dev(inp["k"], cfg, "k"), to_dev(inp["alpha"], cfg, "alpha"),
                            to_dev(inp["theta"], cfg, "theta"), to_dev(inp["beta"], cfg, "beta"), G, Y, M, W, turns,
                            chunk)
    torch.cuda.synchronize()
    cx = lambda t: t.cpu().numpy().astype(np.float64)[..., 0] + 1j * t.cpu().numpy().astype(np.float64)[..., 1]
    G, Y, M, W = cx(G), cx(Y), cx(M), cx(W)
    got_turns = turns.cpu().numpy().view(np.uint32)
    want_turns = np.moveaxis(bookkeeping.cumulative_phase_turns(np.moveaxis(inp["theta"], 1, 2), chunk), 2, 1)
    assert np.array_equal(got_turns, want_turns)
    worst = 0.0
    for b in range(B):
        for h in range(H):
            kc = chunk_wy.pair(inp["k"][b, :, h])
            for c in range(NC):
                sl = slice(c * C, min((c + 1) * C, T))
                L = sl.stop - sl.start
                g, y, w, mm = chunk_wy.chunk_factors(kc[sl], inp["alpha"][b, sl, h].astype(np.float64),
                                                     inp["theta"][b, sl, h].astype(np.float64),
                                                     inp["beta"][b, sl, h].astype(np.float64))
                worst = max(worst, rel_err(G[b, h, c].view(np.float64), g.view(np.float64)),
                            rel_err(Y[b, h, c][:, :L].copy().view(np.float64), y.copy().view(np.float64)),
                            rel_err(W[b, h, c][:, :L].copy().view(np.float64), w.copy().view(np.float64)),
                            rel_err(M[b, h, c][:L, :L].copy().view(np.float64), mm.copy().view(np.float64)))
                # padded tail tokens are neutral: zero columns, identity rows
                assert np.all(Y[b, h, c][:, L:] == 0) and np.all(W[b, h, c][:, L:] == 0)
                assert np.array_equal(M[b, h, c][L:, :], np.eye(C)[L:, :])
                # the product the factors stand for, P = Gamma - Y M W^*, against the oracle's
                P_gpu = np.diag(G[b, h, c]) - Y[b, h, c] @ M[b, h, c] @ W[b, h, c].conj().T
                P_ref = np.diag(g) - y @ mm @ w.conj().T
                assert np.abs(P_gpu - P_ref).max() < 2e-5
    assert worst < 1e-4, worst


@pytest.mark.parametrize("case", ["zeros_and_tiny", "all_one", "strong_everywhere", "one_dead_coordinate"])
@pytest.mark.parametrize("d_k,chunk", [(128, 64), (64, 32)])
def test_chunk_factors_decay_and_write_extremes(case, d_k, chunk):
    """The factor export forms only decay ratios a_t / a_i <= 1 (split at the level boundaries on the tensor cores,
    direct inside the 8-token blocks), so every alpha in [0, 1] is admissible (Section 3 admits alpha = 0): chunks
    with exact zeros, with factors of 1e-6, with alpha = 1 throughout and with strong decay everywhere, beta in
    {0, 1} mixed in and phases far outside (-pi, pi], against the constructive recursion at the usual bar."""
    T, B, H = 2 * chunk + 5, 1, 2
    cfg = workloads.CONFIGS[0].scaled(name="facx", B=B, T=T, H=H, d_k=d_k, chunk=chunk, dtype="bf16", seed=77)
    inp = workloads.forward_inputs(cfg)
    rng = np.random.default_rng([cfg.seed, len(case)])
    m, C = cfg.m, chunk
    alpha = inp["alpha"].copy()
    if case == "zeros_and_tiny":
        pick = rng.random(alpha.shape)
        alpha[pick < 0.05] = 0.0
        alpha[(pick >= 0.05) & (pick < 0.15)] = 1e-6
        alpha[(pick >= 0.15) & (pick < 0.30)] = 1.0
    elif case == "all_one":
        alpha[:] = 1.0
    elif case == "strong_everywhere":
        alpha[:] = (1e-3 * (1.0 + rng.random(alpha.shape))).astype(np.float32)
    else:
        alpha[..., 3] = 0.0                               # one coordinate forgets everything at every token
    beta = inp["beta"].copy()
    pick = rng.random(beta.shape)
    beta[pick < 0.2] = 0.0
    beta[pick > 0.8] = 1.0
    theta = (inp["theta"] * 16.0).astype(np.float32)      # up to about +-50 rad
    NC = -(-T // C)
    G = torch.full((B, H, NC, m, 2), float("nan"), device=DEV)
    Y = torch.full((B, H, NC, m, C, 2), float("nan"), device=DEV)
    M = torch.full((B, H, NC, C, C, 2), float("nan"), device=DEV)
    W = torch.full((B, H, NC, m, C, 2), float("nan"), device=DEV)
    turns = torch.zeros(B, T, H, m, device=DEV, dtype=torch.int32)
    sfda.sfda_chunk_factors(to_dev(inp["k"], cfg, "k"), to_dev(alpha, cfg, "alpha"), to_dev(theta, cfg, "theta"),
                            to_dev(beta, cfg, "beta"), G, Y, M, W, turns, chunk)
    torch.cuda.synchronize()
    cx = lambda t: t.cpu().numpy().astype(np.float64)[..., 0] + 1j * t.cpu().numpy().astype(np.float64)[..., 1]
    G, Y, M, W = cx(G), cx(Y), cx(M), cx(W)
    assert np.isfinite(G).all() and np.isfinite(Y).all() and np.isfinite(M).all() and np.isfinite(W).all()
    want_turns = np.moveaxis(bookkeeping.cumulative_phase_turns(np.moveaxis(theta, 1, 2), chunk), 2, 1)
    assert np.array_equal(turns.cpu().numpy().view(np.uint32), want_turns)
    worst = 0.0
    for h in range(H):
        kc = chunk_wy.pair(inp["k"][0, :, h])
        for c in range(NC):
            sl = slice(c * C, min((c + 1) * C, T))
            L = sl.stop - sl.start
            g, y, w, mm = chunk_wy.chunk_factors(kc[sl], alpha[0, sl, h].astype(np.float64),
                                                 theta[0, sl, h].astype(np.float64), beta[0, sl, h].astype(np.float64))
            # absolute bars: the keys have unit norm, so every factor is O(1) at most and a column that decays to
            # nothing has nothing to be relative to
            worst = max(worst, np.abs(G[0, h, c] - g).max(), np.abs(Y[0, h, c][:, :L] - y).max(),
                        np.abs(W[0, h, c][:, :L] - w).max(), np.abs(M[0, h, c][:L, :L] - mm).max())
            P_gpu = np.diag(G[0, h, c]) - Y[0, h, c] @ M[0, h, c] @ W[0, h, c].conj().T
            assert np.abs(P_gpu - (np.diag(g) - y @ mm @ w.conj().T)).max() < 2e-5
    assert worst < 1e-4, worst


@pytest.mark.parametrize("C,d_k,T,dtype", [(128, 128, 200, "bf16"), (128, 128, 150, "f32"), (128, 64, 128, "f32"),
                                           (128, 128, 64, "bf16"), (128, 64, 333, "bf16"), (256, 128, 512, "bf16"),
                                           (256, 128, 300, "f32"), (256, 64, 700, "bf16"), (256, 128, 130, "f32"),
                                           (256, 64, 64, "f32")])
def test_chunk_factors_of_128_and_256_token_chunks(C, d_k, T, dtype):
    """Factors of chunks of 128 and 256 tokens (Section 6 "Chunk size": C = 64-256; App. E protocol C in {64, 128}),
    which the library composes exactly out of 64-token tiles (block form of Eq. "constructive-M", one tile appended
    per launch), against the constructive recursion run over the whole chunk: full chunks, tiles with a ragged tail,
    chunks whose later tiles are empty, and the chunk-local integer phases."""
    cfg = workloads.CONFIGS[0].scaled(name="fac128", B=2, T=T, H=2, d_k=d_k, chunk=64, dtype=dtype, seed=900 + T)
    inp = workloads.forward_inputs(cfg)
    B, H, m = cfg.B, cfg.H, cfg.m
    NC, tail = sfda.sfda_plan(T, C)
    assert (NC, tail) == bookkeeping.chunk_plan(T, C)
    G = torch.full((B, H, NC, m, 2), float("nan"), device=DEV)
    Y = torch.full((B, H, NC, m, C, 2), float("nan"), device=DEV)
    M = torch.full((B, H, NC, C, C, 2), float("nan"), device=DEV)
    W = torch.full((B, H, NC, m, C, 2), float("nan"), device=DEV)
    turns = torch.zeros(B, T, H, m, device=DEV, dtype=torch.int32)
    sfda.sfda_chunk_factors(to_dev(inp["k"], cfg, "k"), to_dev(inp["alpha"], cfg, "alpha"),
                            to_dev(inp["theta"], cfg, "theta"), to_dev(inp["beta"], cfg, "beta"), G, Y, M, W, turns, C)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == C // 64
    cx = lambda t: t.cpu().numpy().astype(np.float64)[..., 0] + 1j * t.cpu().numpy().astype(np.float64)[..., 1]
    G, Y, M, W = cx(G), cx(Y), cx(M), cx(W)
    want_turns = np.moveaxis(bookkeeping.cumulative_phase_turns(np.moveaxis(inp["theta"], 1, 2), C), 2, 1)
    assert np.array_equal(turns.cpu().numpy().view(np.uint32), want_turns)
    worst = 0.0
    for b in range(B):
        for h in range(H):
            kc = chunk_wy.pair(inp["k"][b, :, h])
            for c in range(NC):
                sl = slice(c * C, min((c + 1) * C, T))
                L = sl.stop - sl.start
                g, y, w, mm = chunk_wy.chunk_factors(kc[sl], inp["alpha"][b, sl, h].astype(np.float64),
                                                     inp["theta"][b, sl, h].astype(np.float64),
                                                     inp["beta"][b, sl, h].astype(np.float64))
                worst = max(worst, rel_err(G[b, h, c].view(np.float64), g.view(np.float64)),
                            rel_err(Y[b, h, c][:, :L].copy().view(np.float64), y.copy().view(np.float64)),
                            rel_err(W[b, h, c][:, :L].copy().view(np.float64), w.copy().view(np.float64)),
                            rel_err(M[b, h, c][:L, :L].copy().view(np.float64), mm.copy().view(np.float64)))
                # padded tail tokens are neutral: zero columns, identity rows; nothing above the diagonal
                assert np.all(Y[b, h, c][:, L:] == 0) and np.all(W[b, h, c][:, L:] == 0)
                assert np.array_equal(M[b, h, c][L:, :], np.eye(C)[L:, :])
                assert np.all(np.triu(M[b, h, c], 1) == 0)
                P_gpu = np.diag(G[b, h, c]) - Y[b, h, c] @ M[b, h, c] @ W[b, h, c].conj().T
                assert np.abs(P_gpu - (np.diag(g) - y @ mm @ w.conj().T)).max() < 2e-5
    assert worst < 1e-4, worst


@pytest.mark.parametrize("chunk", [128, 256])
def test_forward_with_chunks_of_128_and_256_tokens(chunk):
    """A chunk of 128 or 256 tokens runs as an exact superchunk of 64-token tiles (Section 6: chunk transfers compose
    exactly, and the recurrence's result does not depend on where a sequence is cut): same bits as chunk = 64 on the
    tensor-core path and on the CUDA-core path, and the oracle's values."""
    cfg = workloads.CONFIGS[1].scaled(name="sup", B=2, T=4 * 256 + 37, H=3, s0_std=0.02)
    inp = workloads.forward_inputs(cfg)
    o64, oi64, S64 = run_forward(cfg, inp)
    o, oi, S = run_forward(cfg.scaled(chunk=chunk), inp)
    assert np.array_equal(o, o64) and np.array_equal(oi, oi64) and np.array_equal(S, S64)
    pairs = [(0, 0), (1, 2)]
    s = workloads.sequences(inp, pairs)
    w_re, w_im, w_S = recurrence.sfda_recurrence(s["q"], s["k"], s["v"], s["alpha"], s["theta"], s["beta"], s["S0"])
    assert rel_err(np.stack([o[b, :, h] for b, h in pairs]), w_re) <= 2e-2
    assert rel_err(np.stack([S[b, h] for b, h in pairs]), w_S) <= 2e-2
    # CUDA-core path (fp32, d_k = 64)
    cfg32 = workloads.CONFIGS[0].scaled(name="sup32", B=1, T=300, H=2, d_k=64, d_v=64, chunk=32, dtype="f32")
    inp32 = workloads.forward_inputs(cfg32)
    a = run_forward(cfg32.scaled(chunk=64), inp32)
    b_ = run_forward(cfg32.scaled(chunk=chunk), inp32)
    assert all(np.array_equal(x, y) for x, y in zip(a, b_))


def test_other_forward_entry_points_with_chunks_of_128_tokens():
    """The fused forward, the two-level scan, the entry point without allocations and the host-buffer entry point take
    chunk = 128 as the same exact superchunk: bit for bit what they return with chunk = 64."""
    cfg = workloads.CONFIGS[1].scaled(name="sup2", B=2, T=2048, H=3, s0_std=0.02, seed=321)
    inp = workloads.forward_inputs(cfg)
    raw = workloads.forward_raw_inputs(cfg)
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    B, T, H = cfg.B, cfg.T, cfg.H
    new = lambda: (torch.empty(B, T, H, 128, device=DEV, dtype=torch.bfloat16),
                   torch.empty(B, T, H, 128, device=DEV, dtype=torch.bfloat16), torch.empty(B, H, 128, 128, device=DEV))
    same = lambda x, y: all(torch.equal(a, b) for a, b in zip(x, y))
    # fused
    outs = []
    for chunk in (64, 128):
        o, o_im, S, _, _ = run_forward_fused(cfg.scaled(chunk=chunk), raw, PARAM)
        outs.append((o, o_im, S))
    assert all(np.array_equal(a, b) for a, b in zip(*outs))
    # two-level scan (4 slices)
    outs = []
    for chunk in (64, 128):
        o, o_im, S = new()
        ws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(B, T, H, 128, 128, chunk, 1, 4), device=DEV, dtype=torch.uint8)
        sfda.sfda_forward_two_level(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S, chunk, 4, ws)
        assert sfda.sfda_workspace_status(ws) == 0
        outs.append((o, o_im, S))
    assert same(*outs)
    # no allocations
    outs = []
    for chunk in (64, 128):
        o, o_im, S = new()
        sfda.sfda_forward_noalloc(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S, chunk)
        assert sfda.sfda_noalloc_status() == 0
        outs.append((o, o_im, S))
    assert same(*outs)
    # host buffers
    h = {k: (None if v is None else to_dev(v, cfg, k).cpu().pin_memory()) for k, v in inp.items()}
    outs = []
    for chunk in (64, 128):
        oh = torch.empty(B, T, H, 128, dtype=torch.bfloat16).pin_memory()
        oh_im, Sh = torch.empty_like(oh).pin_memory(), torch.empty(B, H, 128, 128).pin_memory()
        arena = torch.empty(sfda.sfda_forward_host_arena_bytes(B, T, H, 128, 128, chunk, 1, True, True, True), device=DEV,
                            dtype=torch.uint8)
        sfda.sfda_forward_host(h["q"], h["k"], h["v"], h["alpha"], h["theta"], h["beta"], h["S0"], oh, oh_im, Sh, chunk, arena)
        torch.cuda.synchronize()
        outs.append((oh.clone(), oh_im.clone(), Sh.clone()))
    assert same(*outs)


# ------------------------------------------------------------------------------------------------
# decode
# ------------------------------------------------------------------------------------------------
def run_decode(cfg, steps, pairs):
    """Run `steps` decode steps on the GPU; keep inputs and outputs of the sampled (b, h) pairs only."""
    from concurrent.futures import ThreadPoolExecutor
    S0 = workloads.decode_initial_state(cfg)
    S = torch.from_numpy(S0).to(DEV)
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    o = torch.empty(cfg.B, cfg.H, cfg.d_v, device=DEV, dtype=dt)
    o_im = torch.empty_like(o)
    bi = torch.tensor([p[0] for p in pairs], device=DEV)
    hi = torch.tensor([p[1] for p in pairs], device=DEV)
    out = torch.empty(steps, len(pairs), cfg.d_v, device=DEV)
    out_im = torch.empty_like(out)
    keys = ("q", "k", "v", "alpha", "theta", "beta")
    sampled = {k: [] for k in keys}
    bsel, hsel = np.array([p[0] for p in pairs]), np.array([p[1] for p in pairs])
    window = 32
    with ThreadPoolExecutor(max_workers=8) as pool:
        for s0 in range(0, steps, window):
            batch = list(pool.map(lambda s: workloads.decode_step_inputs(cfg, s), range(s0, min(s0 + window, steps))))
            for i, x in enumerate(batch):
                for k in keys:
                    sampled[k].append(x[k][bsel, hsel])
                d = {k: to_dev(v, cfg, k) for k, v in x.items()}
                sfda.sfda_step(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], S, o, o_im)
                out[s0 + i] = o[bi, hi].float()
                out_im[s0 + i] = o_im[bi, hi].float()
    torch.cuda.synchronize()
    seqs = {k: np.stack(v, axis=1).astype(np.float64) for k, v in sampled.items()}     # [N, steps, ...]
    S0s = np.stack([S0[b, h] for b, h in pairs]).astype(np.float64)
    S_end = np.stack([S[b, h].cpu().numpy() for b, h in pairs])
    return seqs, S0s, out.cpu().numpy().transpose(1, 0, 2), out_im.cpu().numpy().transpose(1, 0, 2), S_end


def check_decode(cfg, pairs, tol_o, tol_S):
    seqs, S0s, o, o_im, S_end = run_decode(cfg, cfg.steps, pairs)
    w_re, w_im, w_S = recurrence.sfda_recurrence(seqs["q"], seqs["k"], seqs["v"], seqs["alpha"], seqs["theta"],
                                                 seqs["beta"], S0s)
    assert rel_err(o, w_re) <= tol_o
    assert rel_err(o_im, w_im) <= tol_o
    assert rel_err(S_end, w_S) <= tol_S


@pytest.mark.parametrize("d_k,d_v,dtype", [(64, 64, "f32"), (64, 128, "f32"), (128, 64, "bf16"), (128, 128, "f32"),
                                           (128, 128, "bf16")])
def test_step_small(d_k, d_v, dtype):
    cfg = workloads.CONFIGS[4].scaled(name="dec", B=3, H=2, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.5, steps=40)
    # fp32 arithmetic; bf16 storage only rounds o
    check_decode(cfg, all_pairs(cfg), 1e-4 if dtype == "f32" else 5e-3, 1e-4)


def test_step_full_size_decode_config():
    """Configuration 4: B = 256 sequences, H = 32, 1024 consecutive steps; the oracle follows 256
    (batch, head) states through all steps."""
    cfg = workloads.CONFIGS[4]
    # 256 of the 8192 states, spread evenly (one in 32: state index 32 i + (i mod 32) visits every head and, with two
    # CTAs per state and four resident CTAs per SM, every SM of every wave)
    pairs = [divmod(32 * i + (i % 32), cfg.H) for i in range(256)]
    check_decode(cfg, pairs, TOL["bf16"], 1e-4)


def test_iterated_step_equals_forward():
    """Decode step by step == chunked forward on the same tokens."""
    cfg = workloads.CONFIGS[0].scaled(name="it", B=2, T=48, H=2, d_k=128, d_v=128, chunk=16, s0_std=0.3, seed=12)
    inp = workloads.forward_inputs(cfg)
    o_f, o_im_f, S_f = run_forward(cfg, inp)
    S = torch.from_numpy(inp["S0"]).to(DEV)
    o = torch.empty(cfg.B, cfg.H, cfg.d_v, device=DEV)
    o_im = torch.empty_like(o)
    for t in range(cfg.T):
        d = {k: to_dev(np.ascontiguousarray(inp[k][:, t]), cfg, k) for k in ("q", "k", "v", "alpha", "theta", "beta")}
        sfda.sfda_step(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], S, o, o_im)
        assert rel_err(o.cpu().numpy(), o_f[:, t]) < 1e-4
        assert rel_err(o_im.cpu().numpy(), o_im_f[:, t]) < 1e-4
    assert rel_err(S.cpu().numpy(), S_f) < 1e-4


# ------------------------------------------------------------------------------------------------
# host-buffer entry point and argument errors
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("B,T,H", [(2, 256, 2), (2, 5, 1), (3, 130, 3), (9, 67, 1)])
def test_forward_host_matches_device_call(B, T, H):
    """Host buffers in, host buffers out, against the device-pointer call: also where a piece of the batch holds a
    number of (token, head) rows that is not a multiple of four (beta then starts off a 16-byte boundary in the
    caller's array) and where the last piece is shorter than the others."""
    cfg = workloads.CONFIGS[1].scaled(name="host", B=B, T=T, H=H, s0_std=0.1)
    inp = workloads.forward_inputs(cfg)
    o_d, o_im_d, S_d = run_forward(cfg, inp)
    h = {}
    for key, val in inp.items():
        t = torch.from_numpy(np.ascontiguousarray(val))
        if key in ("q", "k", "v"):
            t = t.to(torch.bfloat16)
        h[key] = t.pin_memory()
    o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, dtype=torch.bfloat16).pin_memory()
    o_im = torch.empty_like(o).pin_memory()
    S_T = torch.empty(cfg.B, cfg.H, cfg.d_k, cfg.d_v).pin_memory()
    n = sfda.sfda_forward_host_arena_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, 1, True, True, True)
    arena = torch.empty(n, dtype=torch.uint8, device=DEV)
    h2d, d2h = sfda.sfda_forward_host(h["q"], h["k"], h["v"], h["alpha"], h["theta"], h["beta"], h["S0"], o, o_im,
                                      S_T, cfg.chunk, arena)
    torch.cuda.synchronize()
    assert h2d == sum(h[k].numel() * h[k].element_size() for k in h)
    assert d2h == 2 * o.numel() * 2 + S_T.numel() * 4
    assert np.array_equal(o.float().numpy(), o_d) and np.array_equal(o_im.float().numpy(), o_im_d)
    assert np.array_equal(S_T.numpy(), S_d)


def test_argument_errors_launch_nothing():
    cfg = workloads.CONFIGS[0]
    inp = workloads.forward_inputs(cfg)
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    o = torch.empty(1, cfg.T, cfg.H, cfg.d_v, device=DEV)
    with pytest.raises(sfda.SfdaError) as e:
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], None, o, None, None, 48)
    assert e.value.status == -3
    with pytest.raises(sfda.SfdaError) as e:
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], None, o[..., 1:].reshape(-1)[1:33],
                          None, None, 16)
    assert e.value.status == -4


# ------------------------------------------------------------------------------------------------
# stable parameterisation: as a kernel of its own, and fused into the forward
# ------------------------------------------------------------------------------------------------
PARAM = dict(alpha_min=0.0, alpha_max=1.0, theta_max=float(np.pi), eps=1e-6)


def raw_to_dev(raw, cfg):
    d = {}
    for key, x in raw.items():
        if x is None:
            d[key] = None
            continue
        t = torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
        if key in ("q", "k_raw", "v") and cfg.dtype == "bf16":
            t = t.to(torch.bfloat16)
        d[key] = t
    return d


@pytest.mark.parametrize("d_k,dtype,rows", [(128, "bf16", (2, 37, 3)), (64, "bf16", (1, 130, 2)),
                                            (128, "f32", (1, 65, 5)), (64, "f32", (3, 1, 1))])
@pytest.mark.parametrize("par", [PARAM, dict(alpha_min=0.25, alpha_max=0.875, theta_max=0.5, eps=0.0)])
def test_frontend_matches_oracle(d_k, dtype, rows, par):
    B, T, H = rows
    cfg = workloads.CONFIGS[0].scaled(name="fe", B=B, T=T, H=H, d_k=d_k, d_v=64, dtype=dtype, seed=40 + d_k)
    raw = workloads.forward_raw_inputs(cfg)
    raw["a_raw"][0, 0, 0, :4] = [-100.0, 100.0, -20.0, 20.0]        # saturation of the sigmoid
    raw["b_raw"][0, 0, 0, :4] = [-50.0, 50.0, 0.0, 1e-4]            # and of tanh; tanh near zero
    raw["c_raw"][0, 0, 0] = -90.0
    d = raw_to_dev(raw, cfg)
    al, th = torch.empty_like(d["a_raw"]), torch.empty_like(d["a_raw"])
    be, k = torch.empty_like(d["c_raw"]), torch.empty_like(d["k_raw"])
    sfda.sfda_frontend(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], par["alpha_min"], par["alpha_max"],
                       par["theta_max"], par["eps"], al, th, be, k)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == 1
    w_al, w_th, w_be, w_k = frontend.stable_parameterisation(raw["a_raw"], raw["b_raw"], raw["c_raw"], raw["k_raw"],
                                                             **par)
    # fp32 evaluation of exp / tanh / sqrt: a few ulp of the result's scale
    assert np.abs(al.cpu().numpy() - w_al).max() <= 1e-6
    assert np.abs(th.cpu().numpy() - w_th).max() <= 1e-6 * max(par["theta_max"], 1.0)
    assert np.abs(be.cpu().numpy() - w_be).max() <= 1e-6
    k_tol = 2.0 ** -8 if dtype == "bf16" else 1e-6                  # one bf16 rounding of values <= 1
    assert np.abs(k.float().cpu().numpy() - w_k).max() <= k_tol * np.abs(w_k).max()
    # in place
    sfda.sfda_frontend(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], par["alpha_min"], par["alpha_max"],
                       par["theta_max"], par["eps"], d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"])
    torch.cuda.synchronize()
    assert torch.equal(d["a_raw"], al) and torch.equal(d["b_raw"], th) and torch.equal(d["c_raw"], be)
    assert torch.equal(d["k_raw"], k)


@pytest.mark.parametrize("d_k,dtype,rows", [(128, "bf16", (2, 37, 3)), (64, "f32", (1, 130, 2)), (128, "f32", (1, 65, 5))])
@pytest.mark.parametrize("par", [PARAM, dict(alpha_min=0.25, alpha_max=0.875, theta_max=0.5, eps=1e-3)])
def test_frontend_backward_matches_oracle(d_k, dtype, rows, par):
    """Gradients with respect to the raw inputs of the stable parameterisation; a zero key passes s dk through; the
    outputs may alias the incoming gradients."""
    B, T, H = rows
    cfg = workloads.CONFIGS[0].scaled(name="feb", B=B, T=T, H=H, d_k=d_k, d_v=64, dtype=dtype, seed=45 + d_k)
    raw = workloads.forward_raw_inputs(cfg)
    raw["a_raw"][0, 0, 0, :4] = [-100.0, 100.0, -20.0, 20.0]
    raw["b_raw"][0, 0, 0, :4] = [-50.0, 50.0, 0.0, 1e-4]
    raw["k_raw"][0, 1, 0] = 0.0
    rng = np.random.default_rng([cfg.seed, 3])
    rnd = (lambda x: workloads.bf16_round(x)) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    g_al = rng.standard_normal(raw["a_raw"].shape, dtype=np.float32)
    g_th = rng.standard_normal(raw["a_raw"].shape, dtype=np.float32)
    g_be = rng.standard_normal(raw["c_raw"].shape, dtype=np.float32)
    g_k = rnd(rng.standard_normal(raw["k_raw"].shape, dtype=np.float32))
    d = raw_to_dev(raw, cfg)
    dt = d["k_raw"].dtype
    t = lambda x, ty=torch.float32: torch.from_numpy(np.ascontiguousarray(x)).to(DEV).to(ty)
    ga, gt, gb, gk = t(g_al), t(g_th), t(g_be), t(g_k, dt)
    da, db, dc, dkr = torch.empty_like(ga), torch.empty_like(gt), torch.empty_like(gb), torch.empty_like(gk)
    sfda.sfda_frontend_backward(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], par["alpha_min"], par["alpha_max"],
                                par["theta_max"], par["eps"], ga, gt, gb, gk, da, db, dc, dkr)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == 1
    w = frontend.stable_parameterisation_backward(raw["a_raw"], raw["b_raw"], raw["c_raw"], raw["k_raw"],
                                                  par["alpha_min"], par["alpha_max"], par["theta_max"], par["eps"],
                                                  g_al, g_th, g_be, g_k)
    for got, want, tol in ((da, w[0], 1e-5), (db, w[1], 1e-5), (dc, w[2], 1e-5),
                           (dkr, w[3], 2.0 ** -8 if dtype == "bf16" else 1e-5)):
        assert rel_err(got.float().cpu().numpy(), want) <= tol
    # in place
    sfda.sfda_frontend_backward(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], par["alpha_min"], par["alpha_max"],
                                par["theta_max"], par["eps"], ga, gt, gb, gk, ga, gt, gb, gk)
    torch.cuda.synchronize()
    assert torch.equal(ga, da) and torch.equal(gt, db) and torch.equal(gb, dc) and torch.equal(gk, dkr)


def test_gradients_with_respect_to_raw_inputs_end_to_end():
    """A training step's backward on raw inputs: sfda_frontend, then sfda_backward on its outputs, then
    sfda_frontend_backward -- against the oracle's composition of the same three maps."""
    cfg = workloads.CONFIGS[0].scaled(name="e2eb", B=1, T=96, H=2, d_k=128, d_v=128, dtype="f32", s0_std=0.3, seed=46)
    raw = workloads.forward_raw_inputs(cfg)
    inp = workloads.forward_inputs(cfg)            # q, v, S0 of the same shapes
    par = PARAM
    d = raw_to_dev(raw, cfg)
    q, v, S0 = (to_dev(inp[k], cfg, k) for k in ("q", "v", "S0"))
    al, th = torch.empty_like(d["a_raw"]), torch.empty_like(d["a_raw"])
    be, k = torch.empty_like(d["c_raw"]), torch.empty_like(d["k_raw"])
    sfda.sfda_frontend(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], par["alpha_min"], par["alpha_max"],
                       par["theta_max"], par["eps"], al, th, be, k)
    up = upstream(cfg, 9)
    g = dict(dq=torch.empty_like(q), dk=torch.empty_like(k), dv=torch.empty_like(v), dalpha=torch.empty_like(al),
             dtheta=torch.empty_like(th), dbeta=torch.empty_like(be), dS0=torch.empty_like(S0))
    ws = torch.empty(sfda.sfda_backward_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, 0), dtype=torch.uint8,
                     device=DEV)
    tdev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).to(DEV)
    sfda.sfda_backward(q, k, v, al, th, be, S0, tdev(up["do_re"]), tdev(up["do_im"]), tdev(up["dS_T"]), g["dq"], g["dk"],
                       g["dv"], g["dalpha"], g["dtheta"], g["dbeta"], g["dS0"], ws)
    da, db, dc, dkr = (torch.empty_like(x) for x in (al, th, be, k))
    sfda.sfda_frontend_backward(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], par["alpha_min"], par["alpha_max"],
                                par["theta_max"], par["eps"], g["dalpha"], g["dtheta"], g["dbeta"], g["dk"], da, db, dc,
                                dkr)
    torch.cuda.synchronize()
    w_al, w_th, w_be, w_k = frontend.stable_parameterisation(raw["a_raw"], raw["b_raw"], raw["c_raw"], raw["k_raw"], **par)
    pairs = all_pairs(cfg)
    sel = lambda x: np.stack([x[b, :, h] for b, h in pairs]).astype(np.float64)
    S0n = np.stack([inp["S0"][b, h] for b, h in pairs]).astype(np.float64)
    dST = np.stack([up["dS_T"][b, h] for b, h in pairs]).astype(np.float64)
    wb = backward.sfda_backward(sel(inp["q"]), sel(w_k), sel(inp["v"]), sel(w_al), sel(w_th), sel(w_be), S0n,
                                sel(up["do_re"]), sel(up["do_im"]), dST)
    unsel = lambda x, like: np.stack([x[i] for i in range(len(pairs))]).reshape(cfg.B, cfg.H, *x.shape[1:]).swapaxes(1, 2)
    wr = frontend.stable_parameterisation_backward(raw["a_raw"], raw["b_raw"], raw["c_raw"], raw["k_raw"], par["alpha_min"],
                                                   par["alpha_max"], par["theta_max"], par["eps"], unsel(wb[3], None),
                                                   unsel(wb[4], None), unsel(wb[5], None), unsel(wb[1], None))
    for got, want in zip((da, db, dc, dkr), wr):
        assert rel_err(got.float().cpu().numpy(), want) <= 2e-4


def test_frontend_zero_key_with_zero_eps_stays_zero():
    cfg = workloads.CONFIGS[0].scaled(name="fe0", B=1, T=8, H=2, d_k=128, dtype="bf16", seed=5)
    raw = workloads.forward_raw_inputs(cfg)
    raw["k_raw"][0, 3, 1] = 0.0
    d = raw_to_dev(raw, cfg)
    sfda.sfda_frontend(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], 0.0, 1.0, 1.0, 0.0, d["a_raw"], d["b_raw"],
                       d["c_raw"], d["k_raw"])
    torch.cuda.synchronize()
    k = d["k_raw"].float().cpu().numpy()
    assert np.isfinite(k).all() and np.all(k[0, 3, 1] == 0.0)


def run_forward_fused(cfg, raw, par, want_im=True, want_state=True):
    d = raw_to_dev(raw, cfg)
    B, T, H = d["q"].shape[:3]
    o = torch.empty(B, T, H, cfg.d_v, device=DEV, dtype=d["q"].dtype)
    o_im = torch.empty_like(o) if want_im else None
    S_T = torch.empty(B, H, cfg.d_k, cfg.d_v, device=DEV, dtype=torch.float32) if want_state else None
    ws_bytes = sfda.sfda_forward_fused_workspace_bytes(B, T, H, cfg.d_k, cfg.d_v, cfg.chunk,
                                                       1 if cfg.dtype == "bf16" else 0)
    assert ws_bytes > 0
    ws = torch.empty(ws_bytes, device=DEV, dtype=torch.uint8)
    sfda.sfda_forward_fused(d["q"], d["k_raw"], d["v"], d["a_raw"], d["b_raw"], d["c_raw"], par["alpha_min"],
                            par["alpha_max"], par["theta_max"], par["eps"], d["S0"], o, o_im, S_T, cfg.chunk, ws)
    torch.cuda.synchronize()
    launches = sfda.last_launch_count()
    return (o.float().cpu().numpy(), None if o_im is None else o_im.float().cpu().numpy(),
            None if S_T is None else S_T.cpu().numpy(), launches, ws)


def oracle_fused_pairs(raw, pairs, par):
    """The oracle's front end in float64 on the raw inputs, then the token-by-token recurrence."""
    sel = lambda key: np.stack([raw[key][b, :, h] for b, h in pairs]).astype(np.float64)
    al, th, be, k = frontend.stable_parameterisation(sel("a_raw"), sel("b_raw"), sel("c_raw"), sel("k_raw"), **par)
    S0 = None if raw["S0"] is None else np.stack([raw["S0"][b, h] for b, h in pairs]).astype(np.float64)
    return recurrence.sfda_recurrence(sel("q"), k, sel("v"), al, th, be, S0)


def check_forward_fused(cfg, raw, pairs, par, tol, **kw):
    o, o_im, S_T, launches, ws = run_forward_fused(cfg, raw, par, **kw)
    w_re, w_im, w_S = oracle_fused_pairs(raw, pairs, par)
    errs = {"o_re": rel_err(np.stack([o[b, :, h] for b, h in pairs]), w_re)}
    if o_im is not None:
        errs["o_im"] = rel_err(np.stack([o_im[b, :, h] for b, h in pairs]), w_im)
    if S_T is not None:
        errs["S_T"] = rel_err(np.stack([S_T[b, h] for b, h in pairs]), w_S)
    for name, e in errs.items():
        assert e <= tol, "%s: %s rel err %.3e > %.1e (%s)" % (cfg.name, name, e, tol, errs)
    return launches, ws


@pytest.mark.parametrize("B,T,H", [(1, 64, 1), (2, 200, 3), (1, 1, 2), (3, 1029, 2)])
def test_forward_fused_tensor_core(B, T, H):
    """One launch: the parameterisation runs inside the tensor-core kernel's operand preparation."""
    cfg = workloads.CONFIGS[1].scaled(name="fused", B=B, T=T, H=H, s0_std=0.3, seed=60 + T)
    raw = workloads.forward_raw_inputs(cfg)
    launches, ws = check_forward_fused(cfg, raw, all_pairs(cfg), PARAM, TOL["bf16"])
    assert launches == 1
    assert sfda.sfda_workspace_status(ws) == 0


def test_forward_fused_tensor_core_time_slices_and_narrow_ranges():
    """Enough chunks per sequence for the launcher to cut time slices; alpha in [0.9, 1], small phases."""
    cfg = workloads.CONFIGS[1].scaled(name="fused_q", B=1, T=4096, H=2, s0_std=0.0, seed=61)
    raw = workloads.forward_raw_inputs(cfg)
    raw["a_raw"] -= 3.0                                   # centred logits: alpha spread over the whole range
    par = dict(alpha_min=0.9, alpha_max=1.0, theta_max=0.3, eps=1e-3)
    launches, ws = check_forward_fused(cfg, raw, all_pairs(cfg), par, TOL["bf16"])
    assert launches == 1 and sfda.sfda_workspace_status(ws) == 0


def test_forward_fused_tensor_core_saturated_inputs():
    """Raw inputs far out in the saturating tails, and keys of very different lengths."""
    cfg = workloads.CONFIGS[1].scaled(name="fused_sat", B=1, T=300, H=2, s0_std=0.2, seed=62)
    raw = workloads.forward_raw_inputs(cfg)
    raw["a_raw"][:, ::7] = 60.0                          # alpha = alpha_max
    raw["a_raw"][:, 3::11, :, ::4] = -60.0               # alpha = alpha_min
    raw["b_raw"][:, ::5] *= 40.0                         # theta = +-theta_max
    raw["c_raw"][:, ::3] = 50.0
    raw["c_raw"][:, 1::3] = -50.0
    raw["k_raw"][:, ::2] = workloads.bf16_round(raw["k_raw"][:, ::2] * 1e-3)
    raw["k_raw"][:, 1::4] = workloads.bf16_round(raw["k_raw"][:, 1::4] * 1e3)
    par = dict(alpha_min=0.5, alpha_max=1.0, theta_max=float(np.pi), eps=1e-6)
    check_forward_fused(cfg, raw, all_pairs(cfg), par, TOL["bf16"])


@pytest.mark.parametrize("d_k,d_v,chunk,dtype", [(64, 64, 16, "f32"), (128, 64, 32, "bf16"), (128, 128, 16, "f32")])
def test_forward_fused_other_shapes_stage_through_the_workspace(d_k, d_v, chunk, dtype):
    cfg = workloads.CONFIGS[0].scaled(name="fused_simt", B=2, T=70, H=2, d_k=d_k, d_v=d_v, chunk=chunk,
                                      dtype=dtype, s0_std=0.4, seed=63)
    raw = workloads.forward_raw_inputs(cfg)
    # bf16: the normalised key is rounded to bf16 on its way through the workspace
    launches, _ = check_forward_fused(cfg, raw, all_pairs(cfg), PARAM, 1e-4 if dtype == "f32" else 1e-2)
    assert launches >= 2


def test_forward_fused_equals_frontend_then_forward_on_fp32_keys():
    """The fused kernel against the library's own two-step route at matching precision is not expected to be
    bitwise equal (fast exponentials inside the kernel); both must sit within the bf16 bar of each other."""
    cfg = workloads.CONFIGS[1].scaled(name="fused_vs", B=2, T=512, H=2, s0_std=0.0, seed=64)
    raw = workloads.forward_raw_inputs(cfg)
    o_f, oi_f, S_f, _, _ = run_forward_fused(cfg, raw, PARAM)
    d = raw_to_dev(raw, cfg)
    al, th = torch.empty_like(d["a_raw"]), torch.empty_like(d["a_raw"])
    be, k = torch.empty_like(d["c_raw"]), torch.empty_like(d["k_raw"])
    sfda.sfda_frontend(d["a_raw"], d["b_raw"], d["c_raw"], d["k_raw"], PARAM["alpha_min"], PARAM["alpha_max"],
                       PARAM["theta_max"], PARAM["eps"], al, th, be, k)
    inp = dict(q=raw["q"], k=k.float().cpu().numpy(), v=raw["v"], alpha=al.cpu().numpy(), theta=th.cpu().numpy(),
               beta=be.cpu().numpy(), S0=None)
    o_u, oi_u, S_u = run_forward(cfg, inp)
    assert rel_err(o_f, o_u) <= TOL["bf16"] and rel_err(oi_f, oi_u) <= TOL["bf16"] and rel_err(S_f, S_u) <= TOL["bf16"]


def test_forward_fused_full_size_headline_all_sequences():
    """The headline sizes on raw inputs, in the launch configuration bench.py times for the fused forward;
    the oracle recomputes every (batch, head) sequence end to end.  Also the bound
    ||S_T||_F <= ||S_0||_F + sum_t beta_t ||v_t|| (Prop. "Basic numerical stability",
    with |k_t| <= 1 from the parameterisation)."""
    cfg = workloads.CONFIGS[2]
    raw = workloads.forward_raw_inputs(cfg)
    o, o_im, S_T, launches, ws = run_forward_fused(cfg, raw, PARAM)
    assert launches == 1 and sfda.sfda_workspace_status(ws) == 0
    assert np.isfinite(o).all() and np.isfinite(o_im).all() and np.isfinite(S_T).all()
    check_all_sequences("fused " + cfg.name, all_pairs(cfg), lambda sub: oracle_fused_pairs(raw, sub, PARAM),
                        (o, o_im, S_T), TOL["bf16"])
    beta = 1.0 / (1.0 + np.exp(-raw["c_raw"].astype(np.float64)))
    vnorm = np.linalg.norm(raw["v"].astype(np.float64), axis=-1)
    bound = np.linalg.norm(raw["S0"].astype(np.float64).reshape(cfg.B, cfg.H, -1), axis=-1) \
        + np.sum(beta * vnorm, axis=1)
    assert (np.linalg.norm(S_T.astype(np.float64).reshape(cfg.B, cfg.H, -1), axis=-1) <= bound * (1 + 1e-2)).all()


@pytest.mark.parametrize("d_k,d_v,dtype,par", [
    (128, 128, "bf16", PARAM), (64, 128, "f32", PARAM),
    (128, 64, "f32", dict(alpha_min=0.25, alpha_max=0.875, theta_max=0.5, eps=0.0))])
def test_step_fused_iterated_matches_oracle(d_k, d_v, dtype, par):
    """Decode on raw inputs, token by token, against the oracle's front end followed by its recurrence."""
    cfg = workloads.CONFIGS[0].scaled(name="stepf", B=2, T=40, H=3, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.3,
                                      seed=70 + d_k)
    raw = workloads.forward_raw_inputs(cfg)
    if par["eps"] > 0:
        raw["k_raw"][0, 5, 1] = 0.0                  # a zero key (0 / (0 + eps) = 0; with eps = 0 the map is 0 / 0)
    pairs = all_pairs(cfg)
    w_re, w_im, w_S = oracle_fused_pairs(raw, pairs, par)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    S = torch.from_numpy(raw["S0"]).to(DEV)
    o = torch.empty(cfg.B, cfg.H, cfg.d_v, device=DEV, dtype=dt)
    o_im = torch.empty_like(o)
    got_re, got_im = [], []
    for t in range(cfg.T):
        d = {k: torch.from_numpy(np.ascontiguousarray(raw[k][:, t])).to(DEV) for k in
             ("q", "k_raw", "v", "a_raw", "b_raw", "c_raw")}
        for k in ("q", "k_raw", "v"):
            d[k] = d[k].to(dt)
        sfda.sfda_step_fused(d["q"], d["k_raw"], d["v"], d["a_raw"], d["b_raw"], d["c_raw"], par["alpha_min"],
                             par["alpha_max"], par["theta_max"], par["eps"], S, o, o_im)
        assert sfda.last_launch_count() == 1
        got_re.append(o.float().cpu().numpy())
        got_im.append(o_im.float().cpu().numpy())
    got_re, got_im = np.stack(got_re, 1), np.stack(got_im, 1)          # [B, T, H, d_v]
    tol = 5e-3 if dtype == "bf16" else 1e-4                            # bf16: only the stored outputs are rounded
    assert rel_err(np.stack([got_re[b, :, h] for b, h in pairs]), w_re) <= tol
    assert rel_err(np.stack([got_im[b, :, h] for b, h in pairs]), w_im) <= tol
    assert rel_err(np.stack([S[b, h].cpu().numpy() for b, h in pairs]), w_S) <= 1e-4


# ------------------------------------------------------------------------------------------------
# backward pass
# ------------------------------------------------------------------------------------------------
def run_backward(cfg, inp, up):
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    dt = d["q"].dtype
    B, T, H = d["q"].shape[:3]
    u = {k: (None if v is None else torch.from_numpy(np.ascontiguousarray(v)).to(DEV)) for k, v in up.items()}
    for key in ("do_re", "do_im"):
        if u[key] is not None:
            u[key] = u[key].to(dt)
    out = dict(dq=torch.empty_like(d["q"]), dk=torch.empty_like(d["k"]), dv=torch.empty_like(d["v"]),
               dalpha=torch.empty_like(d["alpha"]), dtheta=torch.empty_like(d["theta"]),
               dbeta=torch.empty_like(d["beta"]),
               dS0=torch.empty(B, H, cfg.d_k, cfg.d_v, device=DEV, dtype=torch.float32))
    n = sfda.sfda_backward_workspace_bytes(B, T, H, cfg.d_k, cfg.d_v, 1 if cfg.dtype == "bf16" else 0)
    blocks = backward_column_blocks(B, H, cfg.d_v)
    shares = blocks * B * T * H if blocks > 1 else 0
    assert n == (B * H * ((T + 63) // 64 + 64) * cfg.d_k * cfg.d_v + shares * 3 * cfg.d_k + (shares + 3) // 4 * 4) * 4
    ws = torch.empty(n, device=DEV, dtype=torch.uint8)
    sfda.sfda_backward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], u["do_re"], u["do_im"],
                       u["dS_T"], out["dq"], out["dk"], out["dv"], out["dalpha"], out["dtheta"], out["dbeta"],
                       out["dS0"], ws)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == (2 if blocks > 1 else 1)   # the sweeps, then the sum of the blocks' shares
    return {k: v.float().cpu().numpy() for k, v in out.items()}


def backward_column_blocks(B, H, d_v):
    """Column blocks per state: the value columns are halved (down to 32 per CTA) while the grid fits 148 SMs."""
    cols = d_v
    while cols > 32 and B * H * (d_v // (cols // 2)) <= 148:
        cols //= 2
    return d_v // cols


def upstream(cfg, seed, want_im=True, want_state=True):
    """Seeded cotangents on the storage grid of the outputs."""
    rng = np.random.default_rng([seed, 99])
    rnd = (lambda x: workloads.bf16_round(x)) if cfg.dtype == "bf16" else (lambda x: x.astype(np.float32))
    return dict(do_re=rnd(rng.standard_normal((cfg.B, cfg.T, cfg.H, cfg.d_v), dtype=np.float32)),
                do_im=rnd(rng.standard_normal((cfg.B, cfg.T, cfg.H, cfg.d_v), dtype=np.float32)) if want_im else None,
                dS_T=rng.standard_normal((cfg.B, cfg.H, cfg.d_k, cfg.d_v), dtype=np.float32) if want_state else None)


def check_backward(cfg, inp, up, pairs, tol):
    got = run_backward(cfg, inp, up)
    s = workloads.sequences(inp, pairs)
    sel = lambda x: None if x is None else np.stack([x[b, :, h] for b, h in pairs]).astype(np.float64)
    dS_T = None if up["dS_T"] is None else np.stack([up["dS_T"][b, h] for b, h in pairs]).astype(np.float64)
    want = backward.sfda_backward(s["q"], s["k"], s["v"], s["alpha"], s["theta"], s["beta"], s["S0"], sel(up["do_re"]),
                                  sel(up["do_im"]), dS_T)
    names = ("dq", "dk", "dv", "dalpha", "dtheta", "dbeta", "dS0")
    errs = {}
    for name, w in zip(names, want):
        g = np.stack([got[name][b, h] for b, h in pairs]) if name == "dS0" else \
            np.stack([got[name][b, :, h] for b, h in pairs])
        errs[name] = rel_err(g, w)
    for name, e in errs.items():
        assert e <= tol, "%s: %s rel err %.3e > %.1e (%s)" % (cfg.name, name, e, tol, errs)
    return errs


@pytest.mark.parametrize("d_k,d_v,T,dtype", [(128, 128, 150, "f32"), (64, 64, 64, "f32"), (128, 64, 65, "bf16"),
                                             (64, 128, 1, "f32"), (128, 128, 200, "bf16")])
def test_backward_matches_oracle(d_k, d_v, T, dtype):
    cfg = workloads.CONFIGS[0].scaled(name="bwd", B=2, T=T, H=2, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.5,
                                      seed=80 + T)
    inp = workloads.forward_inputs(cfg)
    # fp32 arithmetic; bf16 storage rounds the stored dq, dk, dv once (2^-9 relative)
    check_backward(cfg, inp, upstream(cfg, T), all_pairs(cfg), 1e-4 if dtype == "f32" else 5e-3)


@pytest.mark.parametrize("B,H,d_v,blocks", [(5, 8, 128, 2), (19, 8, 128, 1), (10, 8, 64, 1), (3, 3, 64, 2)])
def test_backward_column_blocks(B, H, d_v, blocks):
    """Few sequences split the value columns over more CTAs (shares summed by a second kernel); many do not."""
    assert backward_column_blocks(B, H, d_v) == blocks
    cfg = workloads.CONFIGS[0].scaled(name="bwd_blocks", B=B, T=70, H=H, d_k=64, d_v=d_v, dtype="bf16", s0_std=0.5,
                                      seed=85 + B)
    inp = workloads.forward_inputs(cfg)
    check_backward(cfg, inp, upstream(cfg, B), [(0, 0), (B - 1, H - 1), (B // 2, 1)], 5e-3)


def test_backward_optional_cotangents_and_zero_state():
    cfg = workloads.CONFIGS[0].scaled(name="bwd_opt", B=1, T=130, H=3, d_k=64, d_v=128, s0_std=0.0, seed=81)
    inp = workloads.forward_inputs(cfg)
    check_backward(cfg, inp, upstream(cfg, 1, want_im=False, want_state=False), all_pairs(cfg), 1e-4)


def test_backward_decay_and_write_extremes():
    """alpha with exact zeros, beta in {0, 1}: the adjoint needs no division, so nothing degenerates."""
    cfg = workloads.CONFIGS[0].scaled(name="bwd_edge", B=1, T=96, H=2, d_k=128, d_v=64, alpha="u(0.0,1)",
                                      beta="bernoulli(0.05)", s0_std=1.0, seed=82)
    inp = workloads.forward_inputs(cfg)
    inp["alpha"][:, ::9, :, ::3] = 0.0
    inp["beta"][:, ::4] = 1.0
    check_backward(cfg, inp, upstream(cfg, 2), all_pairs(cfg), 1e-4)


def test_backward_is_deterministic():
    cfg = workloads.CONFIGS[1].scaled(name="bwd_det", B=1, T=192, H=2, s0_std=0.1, seed=83)
    inp, up = workloads.forward_inputs(cfg), None
    up = upstream(cfg, 3)
    a, b = run_backward(cfg, inp, up), run_backward(cfg, inp, up)
    for key in a:
        assert np.array_equal(a[key], b[key]), key


def test_backward_full_size_headline_sampled():
    """The headline sizes, in the launch configuration bench.py times; the oracle recomputes the gradients of a
    sample of (batch, head) sequences end to end.  bf16 storage of dq, dk, dv."""
    cfg = workloads.CONFIGS[2]
    inp = workloads.forward_inputs(cfg)
    pairs = [(0, 0), (cfg.B - 1, cfg.H - 1), (3, 17)]
    check_backward(cfg, inp, upstream(cfg, 4), pairs, 5e-3)


# ------------------------------------------------------------------------------------------------
# two-level scan over time slices
# ------------------------------------------------------------------------------------------------
def run_two_level(cfg, inp, n_slices, want_im=True, want_state=True):
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    B, T, H = d["q"].shape[:3]
    o = torch.empty(B, T, H, cfg.d_v, device=DEV, dtype=d["q"].dtype)
    o_im = torch.empty_like(o) if want_im else None
    S_T = torch.empty(B, H, cfg.d_k, cfg.d_v, device=DEV, dtype=torch.float32) if want_state else None
    n = sfda.sfda_forward_two_level_workspace_bytes(B, T, H, cfg.d_k, cfg.d_v, cfg.chunk, 1, n_slices)
    assert n > 0
    ws = torch.empty(n, device=DEV, dtype=torch.uint8)
    sfda.sfda_forward_two_level(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T,
                                cfg.chunk, n_slices, ws)
    torch.cuda.synchronize()
    launches = sfda.last_launch_count()
    assert sfda.sfda_workspace_status(ws) == 0
    return (o.float().cpu().numpy(), None if o_im is None else o_im.float().cpu().numpy(),
            None if S_T is None else S_T.cpu().numpy(), launches)


@pytest.mark.parametrize("B,T,H,n_slices,s0", [(1, 2048, 2, 2, 0.3), (2, 2048, 1, 4, 0.0), (1, 4096, 3, 8, 0.3), (1, 4096, 2, 16, 0.3),
                                               (1, 2048, 2, 0, 0.3)])
def test_forward_two_level_matches_oracle(B, T, H, n_slices, s0):
    cfg = workloads.CONFIGS[1].scaled(name="two_level", B=B, T=T, H=H, s0_std=s0, seed=90 + n_slices)
    inp = workloads.forward_inputs(cfg)
    pairs = all_pairs(cfg)
    o, o_im, S_T, launches = run_two_level(cfg, inp, n_slices)
    w_re, w_im, w_S = oracle_pairs(inp, pairs)
    assert rel_err(np.stack([o[b, :, h] for b, h in pairs]), w_re) <= TOL["bf16"]
    assert rel_err(np.stack([o_im[b, :, h] for b, h in pairs]), w_im) <= TOL["bf16"]
    assert rel_err(np.stack([S_T[b, h] for b, h in pairs]), w_S) <= TOL["bf16"]
    # two fills, three forward passes, one scan; left to itself the library does not slice two sequences of 32
    # chunks (fewer than four slices cannot pay) and runs the plain forward
    assert launches == (6 if n_slices else 1)


def test_forward_two_level_optional_outputs_and_agreement_with_the_plain_forward():
    cfg = workloads.CONFIGS[1].scaled(name="two_level_opt", B=1, T=4096, H=2, s0_std=0.1, seed=95)
    inp = workloads.forward_inputs(cfg)
    o2, none_im, none_S, _ = run_two_level(cfg, inp, 4, want_im=False, want_state=False)
    assert none_im is None and none_S is None
    o1, _, _ = run_forward(cfg, inp)
    assert rel_err(o2, o1) <= TOL["bf16"]


def test_forward_two_level_long_context_sampled():
    """Configuration 3 (B=1, T=131072, H=16: 16 sequences on 148 SMs) with the library's own choice of slices;
    the oracle recomputes sampled heads end to end."""
    cfg = workloads.CONFIGS[3]
    inp = workloads.forward_inputs(cfg)
    pairs = [(0, 0), (0, 9)]
    o, o_im, S_T, launches = run_two_level(cfg, inp, 0)
    assert launches == 6
    assert np.isfinite(o).all() and np.isfinite(o_im).all() and np.isfinite(S_T).all()
    w_re, w_im, w_S = oracle_pairs(inp, pairs)
    assert rel_err(np.stack([o[b, :, h] for b, h in pairs]), w_re) <= TOL["bf16"]
    assert rel_err(np.stack([o_im[b, :, h] for b, h in pairs]), w_im) <= TOL["bf16"]
    assert rel_err(np.stack([S_T[b, h] for b, h in pairs]), w_S) <= TOL["bf16"]


def test_chunk_factors_full_size_headline_sampled():
    """The factor export at the headline sizes, in the launch configuration bench.py times; the oracle recomputes
    sampled chunks (first, middle, last of sampled sequences), and the phase turns are compared on whole sequences."""
    cfg = workloads.CONFIGS[2]
    inp = workloads.forward_inputs(cfg)
    B, H, m, C, T = cfg.B, cfg.H, cfg.m, cfg.chunk, cfg.T
    NC = T // C
    G = torch.empty(B, H, NC, m, 2, device=DEV)
    Y = torch.empty(B, H, NC, m, C, 2, device=DEV)
    W = torch.empty_like(Y)
    M = torch.empty(B, H, NC, C, C, 2, device=DEV)
    turns = torch.empty(B, T, H, m, device=DEV, dtype=torch.int32)
    sfda.sfda_chunk_factors(to_dev(inp["k"], cfg, "k"), to_dev(inp["alpha"], cfg, "alpha"),
                            to_dev(inp["theta"], cfg, "theta"), to_dev(inp["beta"], cfg, "beta"), G, Y, M, W, turns, C)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == 1
    cx = lambda t: t.cpu().numpy().astype(np.float64)[..., 0] + 1j * t.cpu().numpy().astype(np.float64)[..., 1]
    worst = 0.0
    for b, h in [(0, 0), (B - 1, H - 1), (3, 17)]:
        kc = chunk_wy.pair(inp["k"][b, :, h])
        for c in (0, NC // 2, NC - 1):
            sl = slice(c * C, (c + 1) * C)
            g, y, w, mm = chunk_wy.chunk_factors(kc[sl], inp["alpha"][b, sl, h].astype(np.float64),
                                                 inp["theta"][b, sl, h].astype(np.float64),
                                                 inp["beta"][b, sl, h].astype(np.float64))
            Gc, Yc, Wc, Mc = cx(G[b, h, c]), cx(Y[b, h, c]), cx(W[b, h, c]), cx(M[b, h, c])
            worst = max(worst, rel_err(Gc.view(np.float64), g.view(np.float64)),
                        rel_err(Yc.copy().view(np.float64), y.copy().view(np.float64)),
                        rel_err(Wc.copy().view(np.float64), w.copy().view(np.float64)),
                        rel_err(Mc.copy().view(np.float64), mm.copy().view(np.float64)))
            assert np.abs((np.diag(Gc) - Yc @ Mc @ Wc.conj().T) - (np.diag(g) - y @ mm @ w.conj().T)).max() < 2e-5
        got = turns[b, :, h].cpu().numpy().view(np.uint32)
        want = bookkeeping.cumulative_phase_turns(inp["theta"][b, :, h], C)
        assert np.array_equal(got, want)
    assert worst < 1e-4, worst


@pytest.mark.parametrize("d_k,d_v,dtype", [(128, 128, "bf16"), (64, 128, "f32"), (128, 64, "f32")])
def test_step_decoupled_iterated_matches_oracle(d_k, d_v, dtype):
    """The write-decoupled variant, token by token, against its oracle (Eq. "sfda-decoupled-main"); with r = k and
    eta = beta the kernel reproduces sfda_step bit for bit."""
    from oracle import variants
    cfg = workloads.CONFIGS[0].scaled(name="stepd", B=2, T=40, H=3, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.3,
                                      seed=120 + d_k)
    inp = workloads.forward_inputs(cfg)
    rng = np.random.default_rng([cfg.seed, 5])
    rnd = (lambda x: workloads.bf16_round(x)) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    r = rnd(0.1 * rng.standard_normal((cfg.B, cfg.T, cfg.H, d_k), dtype=np.float32))
    eta = rng.uniform(0.0, 1.0, (cfg.B, cfg.T, cfg.H)).astype(np.float32)
    eta[:, ::7] = 0.0                                   # no erase at all on some tokens
    pairs = all_pairs(cfg)
    sel = lambda x: np.stack([x[b, :, h] for b, h in pairs]).astype(np.float64)
    S0 = np.stack([inp["S0"][b, h] for b, h in pairs]).astype(np.float64)
    w_re, w_im, w_S = variants.sfda_decoupled_recurrence(sel(inp["q"]), sel(inp["k"]), sel(r), sel(inp["v"]),
                                                         sel(inp["alpha"]), sel(inp["theta"]), sel(eta),
                                                         sel(inp["beta"]), S0)
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    S = torch.from_numpy(inp["S0"]).to(DEV)
    S_tied = S.clone()
    o = torch.empty(cfg.B, cfg.H, cfg.d_v, device=DEV, dtype=dt)
    o_im, o2, o2_im = torch.empty_like(o), torch.empty_like(o), torch.empty_like(o)
    got_re, got_im = [], []
    for t in range(cfg.T):
        d = {k: to_dev(np.ascontiguousarray(inp[k][:, t]), cfg, k) for k in ("q", "k", "v", "alpha", "theta", "beta")}
        rt = torch.from_numpy(np.ascontiguousarray(r[:, t])).to(DEV).to(dt)
        et = torch.from_numpy(np.ascontiguousarray(eta[:, t])).to(DEV)
        sfda.sfda_step_decoupled(d["q"], d["k"], rt, d["v"], d["alpha"], d["theta"], et, d["beta"], S, o, o_im)
        assert sfda.last_launch_count() == 1
        got_re.append(o.float().cpu().numpy())
        got_im.append(o_im.float().cpu().numpy())
        # r = k, eta = beta: the tied step
        S_a = S_tied.clone()
        sfda.sfda_step_decoupled(d["q"], d["k"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["beta"], S_a, o2,
                                 o2_im)
        sfda.sfda_step(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], S_tied, o, o_im)
        assert rel_err(S_a.cpu().numpy(), S_tied.cpu().numpy()) < 1e-6 and rel_err(o2.float().cpu().numpy(), o.float().cpu().numpy()) < 1e-2
    got_re, got_im = np.stack(got_re, 1), np.stack(got_im, 1)
    tol = 5e-3 if dtype == "bf16" else 1e-4
    assert rel_err(np.stack([got_re[b, :, h] for b, h in pairs]), w_re) <= tol
    assert rel_err(np.stack([got_im[b, :, h] for b, h in pairs]), w_im) <= tol
    assert rel_err(np.stack([S[b, h].cpu().numpy() for b, h in pairs]), w_S) <= 1e-4


@pytest.mark.parametrize("d_k,d_v,T,dtype", [(128, 128, 150, "f32"), (64, 64, 33, "f32"), (128, 64, 200, "bf16"),
                                             (64, 128, 1, "f32")])
def test_forward_decoupled_matches_oracle(d_k, d_v, T, dtype):
    """The write-decoupled variant over whole sequences against its oracle; with r = k and eta = beta it agrees with
    the tied forward of the library."""
    from oracle import variants
    cfg = workloads.CONFIGS[0].scaled(name="fwdd", B=2, T=T, H=2, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.4,
                                      seed=130 + T)
    inp = workloads.forward_inputs(cfg)
    rng = np.random.default_rng([cfg.seed, 6])
    rnd = (lambda x: workloads.bf16_round(x)) if dtype == "bf16" else (lambda x: x.astype(np.float32))
    r = rnd(0.1 * rng.standard_normal((cfg.B, T, cfg.H, d_k), dtype=np.float32))
    eta = rng.uniform(0.0, 1.0, (cfg.B, T, cfg.H)).astype(np.float32)
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    dt = d["q"].dtype
    rt, et = torch.from_numpy(r).to(DEV).to(dt), torch.from_numpy(eta).to(DEV)
    o = torch.empty(cfg.B, T, cfg.H, d_v, device=DEV, dtype=dt)
    o_im = torch.empty_like(o)
    S_T = torch.empty(cfg.B, cfg.H, d_k, d_v, device=DEV)
    sfda.sfda_forward_decoupled(d["q"], d["k"], rt, d["v"], d["alpha"], d["theta"], et, d["beta"], d["S0"], o, o_im, S_T)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == 1
    pairs = all_pairs(cfg)
    sel = lambda x: np.stack([x[b, :, h] for b, h in pairs]).astype(np.float64)
    S0 = np.stack([inp["S0"][b, h] for b, h in pairs]).astype(np.float64)
    w_re, w_im, w_S = variants.sfda_decoupled_recurrence(sel(inp["q"]), sel(inp["k"]), sel(r), sel(inp["v"]),
                                                         sel(inp["alpha"]), sel(inp["theta"]), sel(eta),
                                                         sel(inp["beta"]), S0)
    tol = 5e-3 if dtype == "bf16" else 1e-4
    on, oin, Sn = o.float().cpu().numpy(), o_im.float().cpu().numpy(), S_T.cpu().numpy()
    assert rel_err(np.stack([on[b, :, h] for b, h in pairs]), w_re) <= tol
    assert rel_err(np.stack([oin[b, :, h] for b, h in pairs]), w_im) <= tol
    assert rel_err(np.stack([Sn[b, h] for b, h in pairs]), w_S) <= 1e-4
    # tied special case against the library's own forward
    sfda.sfda_forward_decoupled(d["q"], d["k"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["beta"], d["S0"],
                                o, None, S_T)
    torch.cuda.synchronize()
    o_t, _, S_t = run_forward(cfg, inp, simt=True)
    assert rel_err(o.float().cpu().numpy(), o_t) <= tol and rel_err(S_T.cpu().numpy(), S_t) <= 1e-4


def _block_case(cfg, seed, flips=True):
    """Write direction, erase strength and reflection flags for the block-control variant."""
    rng = np.random.default_rng([cfg.seed, seed])
    rnd = (lambda x: workloads.bf16_round(x)) if cfg.dtype == "bf16" else (lambda x: x.astype(np.float32))
    r = rnd(0.1 * rng.standard_normal((cfg.B, cfg.T, cfg.H, cfg.d_k), dtype=np.float32))
    eta = rng.uniform(0.0, 1.0, (cfg.B, cfg.T, cfg.H)).astype(np.float32)
    flip = (rng.uniform(size=(cfg.B, cfg.T, cfg.H, cfg.d_k // 2)) < 0.3).astype(np.uint8) if flips else None
    return r, eta, flip


@pytest.mark.parametrize("d_k,d_v,T,dtype,erase", [(128, 128, 90, "f32", 1), (64, 64, 33, "f32", 0),
                                                   (128, 64, 120, "bf16", 1), (64, 128, 1, "f32", 0)])
def test_forward_blocks_matches_oracle(d_k, d_v, T, dtype, erase):
    """2 x 2 rotation / reflection control blocks with the complex or the real rank-one erase (Eq. "intro-sfda-real")
    against the dense real-matrix oracle; without reflections and with the complex erase the kernel reproduces
    sfda_forward_decoupled bit for bit."""
    from oracle import variants
    cfg = workloads.CONFIGS[0].scaled(name="fwdb", B=2, T=T, H=2, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.4,
                                      seed=140 + T)
    inp = workloads.forward_inputs(cfg)
    r, eta, flip = _block_case(cfg, 7)
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    dt = d["q"].dtype
    rt, et, ft = torch.from_numpy(r).to(DEV).to(dt), torch.from_numpy(eta).to(DEV), torch.from_numpy(flip).to(DEV)
    o = torch.empty(cfg.B, T, cfg.H, d_v, device=DEV, dtype=dt)
    o_im = torch.empty_like(o)
    S_T = torch.empty(cfg.B, cfg.H, d_k, d_v, device=DEV)
    sfda.sfda_forward_blocks(d["q"], d["k"], rt, d["v"], d["alpha"], d["theta"], ft, et, d["beta"], d["S0"], o, o_im,
                             S_T, erase)
    torch.cuda.synchronize()
    assert sfda.last_launch_count() == 1
    pairs = all_pairs(cfg)
    sel = lambda x: np.stack([x[b, :, h] for b, h in pairs]).astype(np.float64)
    S0 = np.stack([inp["S0"][b, h] for b, h in pairs]).astype(np.float64)
    w_re, w_im, w_S = variants.sfda_block_control_recurrence(sel(inp["q"]), sel(inp["k"]), sel(r), sel(inp["v"]),
                                                             sel(inp["alpha"]), sel(inp["theta"]), sel(flip), sel(eta),
                                                             sel(inp["beta"]), S0, real_erase=bool(erase))
    tol = 5e-3 if dtype == "bf16" else 1e-4
    on, oin, Sn = o.float().cpu().numpy(), o_im.float().cpu().numpy(), S_T.cpu().numpy()
    assert rel_err(np.stack([on[b, :, h] for b, h in pairs]), w_re) <= tol
    assert rel_err(np.stack([oin[b, :, h] for b, h in pairs]), w_im) <= tol
    assert rel_err(np.stack([Sn[b, h] for b, h in pairs]), w_S) <= 1e-4
    # no reflections, complex erase: the write-decoupled forward
    o2, o2_im, S2 = torch.empty_like(o), torch.empty_like(o), torch.empty_like(S_T)
    sfda.sfda_forward_blocks(d["q"], d["k"], rt, d["v"], d["alpha"], d["theta"], None, et, d["beta"], d["S0"], o, o_im,
                             S_T, sfda.ERASE_COMPLEX)
    sfda.sfda_forward_decoupled(d["q"], d["k"], rt, d["v"], d["alpha"], d["theta"], et, d["beta"], d["S0"], o2, o2_im, S2)
    torch.cuda.synchronize()
    assert torch.equal(o, o2) and torch.equal(o_im, o2_im) and torch.equal(S_T, S2)


@pytest.mark.parametrize("d_k,d_v,dtype,erase", [(128, 128, "bf16", 1), (64, 128, "f32", 0), (128, 64, "f32", 1)])
def test_step_blocks_iterated_matches_oracle(d_k, d_v, dtype, erase):
    """The decode step of the block-control variant, token by token, against the dense real-matrix oracle."""
    from oracle import variants
    cfg = workloads.CONFIGS[0].scaled(name="stepb", B=2, T=24, H=3, d_k=d_k, d_v=d_v, dtype=dtype, s0_std=0.3,
                                      seed=150 + d_k)
    inp = workloads.forward_inputs(cfg)
    r, eta, flip = _block_case(cfg, 8)
    pairs = all_pairs(cfg)
    sel = lambda x: np.stack([x[b, :, h] for b, h in pairs]).astype(np.float64)
    S0 = np.stack([inp["S0"][b, h] for b, h in pairs]).astype(np.float64)
    w_re, w_im, w_S = variants.sfda_block_control_recurrence(sel(inp["q"]), sel(inp["k"]), sel(r), sel(inp["v"]),
                                                             sel(inp["alpha"]), sel(inp["theta"]), sel(flip), sel(eta),
                                                             sel(inp["beta"]), S0, real_erase=bool(erase))
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    S = torch.from_numpy(inp["S0"]).to(DEV)
    o = torch.empty(cfg.B, cfg.H, cfg.d_v, device=DEV, dtype=dt)
    o_im = torch.empty_like(o)
    got_re, got_im = [], []
    for t in range(cfg.T):
        d = {k: to_dev(np.ascontiguousarray(inp[k][:, t]), cfg, k) for k in ("q", "k", "v", "alpha", "theta", "beta")}
        rt = torch.from_numpy(np.ascontiguousarray(r[:, t])).to(DEV).to(dt)
        et = torch.from_numpy(np.ascontiguousarray(eta[:, t])).to(DEV)
        ft = torch.from_numpy(np.ascontiguousarray(flip[:, t])).to(DEV)
        sfda.sfda_step_blocks(d["q"], d["k"], rt, d["v"], d["alpha"], d["theta"], ft, et, d["beta"], S, o, o_im, erase)
        assert sfda.last_launch_count() == 1
        got_re.append(o.float().cpu().numpy())
        got_im.append(o_im.float().cpu().numpy())
    got_re, got_im = np.stack(got_re, 1), np.stack(got_im, 1)
    tol = 5e-3 if dtype == "bf16" else 1e-4
    assert rel_err(np.stack([got_re[b, :, h] for b, h in pairs]), w_re) <= tol
    assert rel_err(np.stack([got_im[b, :, h] for b, h in pairs]), w_im) <= tol
    assert rel_err(np.stack([S[b, h].cpu().numpy() for b, h in pairs]), w_S) <= 1e-4


def test_blocks_track_dihedral_groups_exactly():
    """Theorem "Dihedral phase-orientation memory" on the device: beta = eta = 0, alpha = 1, every row pair j of a
    state starts as the 2 x 2 identity in columns (2j, 2j+1) and is driven by its own random word in R (rotation by
    2 pi / 7), F (reflection), RF; the final block is rho of the product, which integer arithmetic in D_7 gives."""
    n, T, B, H, d_k, d_v = 7, 50, 1, 2, 64, 64
    m = d_k // 2
    rng = np.random.default_rng(160)
    sym = rng.integers(0, 3, (B, T, H, m))
    theta = np.where(sym == 1, 0.0, 2 * np.pi / n).astype(np.float32)
    flip = (sym >= 1).astype(np.uint8)
    S0 = np.zeros((B, H, d_k, d_v), np.float32)
    for j in range(m):
        S0[:, :, 2 * j, 2 * j] = 1.0
        S0[:, :, 2 * j + 1, 2 * j + 1] = 1.0
    z = lambda *shape: torch.zeros(*shape, device=DEV)
    o, o_im = z(B, T, H, d_v), z(B, T, H, d_v)
    S_T = torch.empty(B, H, d_k, d_v, device=DEV)
    sfda.sfda_forward_blocks(z(B, T, H, d_k), z(B, T, H, d_k), z(B, T, H, d_k), z(B, T, H, d_v),
                             torch.ones(B, T, H, m, device=DEV), torch.from_numpy(theta).to(DEV),
                             torch.from_numpy(flip).to(DEV), z(B, T, H), z(B, T, H), torch.from_numpy(S0).to(DEV), o,
                             o_im, S_T, sfda.ERASE_REAL)
    torch.cuda.synchronize()
    got = S_T.cpu().numpy().astype(np.float64)
    want = np.zeros_like(got)
    for h in range(H):
        for j in range(m):
            a, f = 0, 0
            for s in sym[0, :, h, j]:
                b_, g = (1, 0) if s == 0 else (0, 1) if s == 1 else (1, 1)
                a, f = (b_ + (-1) ** g * a) % n, (g + f) % 2
            ang = 2 * np.pi * a / n
            R = np.array([[np.cos(ang), -np.sin(ang)], [np.sin(ang), np.cos(ang)]])
            want[0, h, 2 * j:2 * j + 2, 2 * j:2 * j + 2] = R @ (np.diag([1.0, -1.0]) if f else np.eye(2))
    assert np.abs(got - want).max() < 2e-5
    off = np.ones((d_k, d_v), bool)
    for j in range(m):
        off[2 * j:2 * j + 2, 2 * j:2 * j + 2] = False
    assert np.count_nonzero(got[:, :, off]) == 0             # nothing leaks out of a pair's own block


def test_final_state_may_alias_the_initial_state():
    """S_T == S0 (the same buffer) is allowed: the plain tensor-core forward and the two-level scan."""
    cfg = workloads.CONFIGS[1].scaled(name="alias", B=2, T=2048, H=2, s0_std=0.3, seed=140)
    inp = workloads.forward_inputs(cfg)
    pairs = all_pairs(cfg)
    _, _, w_S = oracle_pairs(inp, pairs)
    d = {k: to_dev(v, cfg, k) for k, v in inp.items()}
    o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, device=DEV, dtype=torch.bfloat16)
    for two_level in (False, True):
        S = d["S0"].clone()
        if two_level:
            ws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk,
                                                                         1, 4), device=DEV, dtype=torch.uint8)
            sfda.sfda_forward_two_level(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], S, o, None, S,
                                        cfg.chunk, 4, ws)
        else:
            ws = torch.empty(sfda.sfda_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, 1),
                             device=DEV, dtype=torch.uint8)
            sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], S, o, None, S, cfg.chunk, ws)
        torch.cuda.synchronize()
        assert rel_err(np.stack([S.cpu().numpy()[b, h] for b, h in pairs]), w_S) <= TOL["bf16"]


def test_more_than_2_to_the_31_elements_per_array():
    """B = 72 at the headline shapes: q, k, v, o hold 2.4e9 elements each, so any 32-bit index arithmetic would
    wrap.  The kernels are deterministic and sequences independent, so the last two batch elements computed inside
    the big batch must equal, bit for bit, the same ones computed alone (forward and fused forward on the tensor
    cores, the backward pass)."""
    import gc
    gc.collect()
    torch.cuda.empty_cache()                       # earlier tests' cached blocks count as used otherwise
    free, _ = torch.cuda.mem_get_info()
    if free < 120e9:
        pytest.skip("needs about 110 GB of free device memory")
    B, T, H, d = 72, 8192, 32, 128
    g = torch.Generator(device=DEV)
    g.manual_seed(7)
    rn = lambda *s: torch.randn(*s, device=DEV, generator=g)
    q, v = rn(B, T, H, d).to(torch.bfloat16), rn(B, T, H, d).to(torch.bfloat16)
    k = rn(B, T, H, d)
    k = (k / k.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
    alpha = torch.sigmoid(3.0 + rn(B, T, H, d // 2))
    theta = (torch.rand(B, T, H, d // 2, device=DEV, generator=g) * 2 - 1) * np.pi
    beta = torch.sigmoid(rn(B, T, H))
    S0 = 0.02 * rn(B, H, d, d)
    ins = (q, k, v, alpha, theta, beta, S0)
    tail = tuple(x[B - 2:].contiguous() for x in ins)

    def forward(x, fused):
        b = x[0].shape[0]
        o = torch.empty(b, T, H, d, device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.empty_like(o), torch.empty(b, H, d, d, device=DEV)
        if fused:      # the same arrays read as raw inputs of the stable parameterisation
            ws = torch.empty(sfda.sfda_forward_fused_workspace_bytes(b, T, H, d, d, 64, 1), dtype=torch.uint8, device=DEV)
            sfda.sfda_forward_fused(x[0], x[1], x[2], x[3], x[4], x[5], 0.0, 1.0, float(np.pi), 1e-6, x[6], o, o_im, S_T,
                                    64, ws)
        else:
            ws = torch.empty(sfda.sfda_workspace_bytes(b, T, H, d, d, 64, 1), dtype=torch.uint8, device=DEV)
            sfda.sfda_forward(*x, o, o_im, S_T, 64, ws)
        torch.cuda.synchronize()
        assert sfda.sfda_workspace_status(ws) == 0
        return o, o_im, S_T

    for fused in (False, True):
        big, small = forward(ins, fused), forward(tail, fused)
        for a, b_ in zip(big, small):
            assert torch.equal(a[B - 2:], b_), "fused" if fused else "plain"
        del big, small
    # backward: cotangents = the inputs themselves (any values do)
    def backward_(x):
        b = x[0].shape[0]
        out = [torch.empty_like(t) for t in x]
        ws = torch.empty(sfda.sfda_backward_workspace_bytes(b, T, H, d, d, 1), dtype=torch.uint8, device=DEV)
        sfda.sfda_backward(*x, x[2], x[0], x[6], *out, ws)
        torch.cuda.synchronize()
        return out
    big, small = backward_(ins), backward_(tuple(x[B - 4:].contiguous() for x in ins))
    for a, b_ in zip(big, small):
        assert torch.equal(a[B - 4:], b_)


def test_more_than_2_to_the_31_elements_other_kernels():
    """The same check for the other kernels: stand-alone parameterisation, factor export, write-decoupled forward
    (B = 72 at the headline shapes), the decode step on 163840 states (2.7e9 state elements) and the two-level scan on
    one batch element of 2^20 tokens, each against the same computation on a small part of the data."""
    import gc
    gc.collect()
    torch.cuda.empty_cache()                       # earlier tests' cached blocks count as used otherwise
    free, _ = torch.cuda.mem_get_info()
    if free < 120e9:
        pytest.skip("needs about 100 GB of free device memory")
    B, T, H, d = 72, 8192, 32, 128
    g = torch.Generator(device=DEV)
    g.manual_seed(8)
    rn = lambda *s: torch.randn(*s, device=DEV, generator=g)
    k = rn(B, T, H, d).to(torch.bfloat16)
    a, b, c = 3.0 + rn(B, T, H, d // 2), rn(B, T, H, d // 2), rn(B, T, H)

    def frontend(x):
        outs = (torch.empty_like(x[0]), torch.empty_like(x[1]), torch.empty_like(x[2]), torch.empty_like(x[3]))
        sfda.sfda_frontend(x[0], x[1], x[2], x[3], 0.0, 1.0, float(np.pi), 1e-6, *outs)
        torch.cuda.synchronize()
        return outs
    big = frontend((a, b, c, k))
    small = frontend(tuple(x[B - 2:].contiguous() for x in (a, b, c, k)))
    for x, y in zip(big, small):
        assert torch.equal(x[B - 2:], y)
    alpha, theta, beta, kn = big
    del a, b, c, small

    def factors(x):
        bb, NC = x[0].shape[0], T // 64
        Gm = torch.empty(bb, H, NC, d // 2, 2, device=DEV)
        Y = torch.empty(bb, H, NC, d // 2, 64, 2, device=DEV)
        W, M = torch.empty_like(Y), torch.empty(bb, H, NC, 64, 64, 2, device=DEV)
        turns = torch.empty(bb, T, H, d // 2, device=DEV, dtype=torch.int32)
        sfda.sfda_chunk_factors(x[0], x[1], x[2], x[3], Gm, Y, M, W, turns, 64)
        torch.cuda.synchronize()
        return Gm, Y, M, W, turns
    big = factors((kn, alpha, theta, beta))
    small = factors(tuple(x[B - 1:].contiguous() for x in (kn, alpha, theta, beta)))
    for x, y in zip(big, small):
        assert torch.equal(x[B - 1:], y)
    del big, small

    q, v = rn(B, T, H, d).to(torch.bfloat16), rn(B, T, H, d).to(torch.bfloat16)
    r, eta = (0.1 * rn(B, T, H, d)).to(torch.bfloat16), torch.rand(B, T, H, device=DEV, generator=g)

    def decoupled(x):
        bb = x[0].shape[0]
        o = torch.empty(bb, T, H, d, device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.empty_like(o), torch.empty(bb, H, d, d, device=DEV)
        sfda.sfda_forward_decoupled(*x, None, o, o_im, S_T)
        torch.cuda.synchronize()
        return o, o_im, S_T
    ins = (q, kn, r, v, alpha, theta, eta, beta)
    big, small = decoupled(ins), decoupled(tuple(x[B - 1:].contiguous() for x in ins))
    for x, y in zip(big, small):
        assert torch.equal(x[B - 1:], y)
    del big, small, ins, q, v, r, eta, kn, alpha, theta, beta, k

    # decode: 4096 x 40 states
    Bd, Hd = 4096, 40
    S = 0.02 * rn(Bd, Hd, d, d)
    qd, vd = rn(Bd, Hd, d).to(torch.bfloat16), rn(Bd, Hd, d).to(torch.bfloat16)
    kd = rn(Bd, Hd, d)
    kd = (kd / kd.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
    ad, td, bd = torch.sigmoid(3.0 + rn(Bd, Hd, d // 2)), rn(Bd, Hd, d // 2), torch.sigmoid(rn(Bd, Hd))
    S_small = S[Bd - 3:].clone()
    o, o_im = torch.empty_like(vd), torch.empty_like(vd)
    sfda.sfda_step(qd, kd, vd, ad, td, bd, S, o, o_im)
    o_s, o_im_s = torch.empty_like(vd[Bd - 3:]), torch.empty_like(vd[Bd - 3:])
    sfda.sfda_step(*(x[Bd - 3:].contiguous() for x in (qd, kd, vd, ad, td, bd)), S_small, o_s, o_im_s)
    torch.cuda.synchronize()
    assert torch.equal(S[Bd - 3:], S_small) and torch.equal(o[Bd - 3:], o_s) and torch.equal(o_im[Bd - 3:], o_im_s)
    del S, S_small, qd, kd, vd, ad, td, bd

    # two-level scan: one batch element, 16 heads, 2^20 tokens (2^31 elements in q); head 15 alone for comparison
    Tl, Hl = 1 << 20, 16
    ql, vl = rn(1, Tl, Hl, d).to(torch.bfloat16), rn(1, Tl, Hl, d).to(torch.bfloat16)
    kl = rn(1, Tl, Hl, d)
    kl = (kl / kl.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
    al, tl, bl = torch.sigmoid(3.0 + rn(1, Tl, Hl, d // 2)), rn(1, Tl, Hl, d // 2), torch.sigmoid(rn(1, Tl, Hl))

    def two_level(x):
        hh = x[0].shape[2]
        o = torch.empty(1, Tl, hh, d, device=DEV, dtype=torch.bfloat16)
        o_im, S_T = torch.empty_like(o), torch.empty(1, hh, d, d, device=DEV)
        ws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(1, Tl, hh, d, d, 64, 1, 8), dtype=torch.uint8,
                         device=DEV)
        sfda.sfda_forward_two_level(*x, None, o, o_im, S_T, 64, 8, ws)
        torch.cuda.synchronize()
        assert sfda.sfda_workspace_status(ws) == 0
        return o, o_im, S_T
    ins = (ql, kl, vl, al, tl, bl)
    big, small = two_level(ins), two_level(tuple(x[:, :, Hl - 1:].contiguous() for x in ins))
    assert torch.equal(big[0][:, :, Hl - 1:], small[0]) and torch.equal(big[1][:, :, Hl - 1:], small[1])
    assert torch.equal(big[2][:, Hl - 1:], small[2])


def test_calls_can_be_captured_in_a_cuda_graph():
    """The library only enqueues on the caller's stream (no allocation, no synchronisation), so its calls can be
    recorded into a CUDA graph and replayed: eight decode steps, a forward, a fused forward, a two-level forward and
    a backward pass give the same bits replayed as run directly."""
    cfg = workloads.CONFIGS[1].scaled(name="graph", B=1, T=4096, H=4, s0_std=0.05, seed=97)
    inp = workloads.forward_inputs(cfg)
    d = {k: to_dev(v, cfg, k) for k, v in inp.items()}
    B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v
    new = lambda *s, dt=torch.bfloat16: torch.empty(*s, device=DEV, dtype=dt)
    o, o_im, S_T = new(B, T, H, dv), new(B, T, H, dv), new(B, H, dk, dv, dt=torch.float32)
    o2, o2_im, S2 = new(B, T, H, dv), new(B, T, H, dv), new(B, H, dk, dv, dt=torch.float32)
    o3, o3_im, S3 = new(B, T, H, dv), new(B, T, H, dv), new(B, H, dk, dv, dt=torch.float32)
    ws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(B, T, H, dk, dv, 64, 1, 4), dtype=torch.uint8, device=DEV)
    ws2 = torch.empty_like(ws)
    ws3 = torch.empty_like(ws)
    grads = [torch.empty_like(d[k]) for k in ("q", "k", "v", "alpha", "theta", "beta")] + [torch.empty_like(S_T)]
    bws = torch.empty(sfda.sfda_backward_workspace_bytes(B, T, H, dk, dv, 1), dtype=torch.uint8, device=DEV)
    S_dec = d["S0"].clone()
    od, od_im = new(B, H, dv), new(B, H, dv)
    step_in = [{k: d[k][:, t].clone() for k in ("q", "k", "v", "alpha", "theta", "beta")} for t in range(8)]

    def work():
        sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, 64, ws)
        sfda.sfda_forward_fused(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], 0.0, 1.0, float(np.pi), 1e-6,
                                d["S0"], o2, o2_im, S2, 64, ws2)
        sfda.sfda_forward_two_level(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o3, o3_im, S3,
                                    64, 4, ws3)
        sfda.sfda_backward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, *grads, bws)
        for x in step_in:
            sfda.sfda_step(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], S_dec, od, od_im)

    outs = [o, o_im, S_T, o2, o2_im, S2, o3, o3_im, S3, S_dec, od, od_im] + grads
    work()
    torch.cuda.synchronize()
    want = [x.clone() for x in outs]
    for x in outs:
        x.zero_()
    S_dec.copy_(d["S0"])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        work()
    for x in outs:                      # capturing runs nothing
        x.zero_()
    S_dec.copy_(d["S0"])
    graph.replay()
    torch.cuda.synchronize()
    assert sfda.sfda_workspace_status(ws) == 0 and sfda.sfda_workspace_status(ws2) == 0
    for got, w in zip(outs, want):
        assert torch.equal(got, w)


def test_concurrent_calls_from_host_threads():
    """Four host threads, each with its own stream, buffers and workspace, call the tensor-core forward 20 times
    at once (the binding releases the interpreter lock during a call): every result equals the serial one bit for
    bit, and no bounded device-side wait runs out although the persistent kernels compete for the SMs."""
    import threading
    d = 128

    def make(seed, B, T, H):
        g = torch.Generator(device=DEV)
        g.manual_seed(seed)
        rn = lambda *s: torch.randn(*s, device=DEV, generator=g)
        q, v = rn(B, T, H, d).to(torch.bfloat16), rn(B, T, H, d).to(torch.bfloat16)
        k = rn(B, T, H, d)
        k = (k / k.norm(dim=-1, keepdim=True)).to(torch.bfloat16)
        a = torch.sigmoid(3.0 + rn(B, T, H, d // 2))
        b = (torch.rand(B, T, H, d // 2, device=DEV, generator=g) * 2 - 1) * np.pi
        return (q, k, v, a, b, torch.sigmoid(rn(B, T, H)), 0.02 * rn(B, H, d, d))

    def run(x, reps):
        B, T, H = x[0].shape[:3]
        stream, outs = torch.cuda.Stream(), []
        with torch.cuda.stream(stream):
            for _ in range(reps):
                o = torch.empty(B, T, H, d, device=DEV, dtype=torch.bfloat16)
                o_im, S_T = torch.empty_like(o), torch.empty(B, H, d, d, device=DEV)
                ws = torch.empty(sfda.sfda_workspace_bytes(B, T, H, d, d, 64, 1), dtype=torch.uint8, device=DEV)
                sfda.sfda_forward(*x, o, o_im, S_T, 64, ws, stream)
                outs.append((o, o_im, S_T, ws))
            stream.synchronize()
        return outs

    torch.cuda.synchronize()
    xs = [make(1, 2, 2048, 16), make(2, 1, 4096, 40), make(3, 4, 1024, 8), make(4, 3, 1536 + 7, 11)]
    serial = [run(x, 1)[0] for x in xs]
    res = [None] * len(xs)

    def worker(i):
        res[i] = run(xs[i], 20)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(xs))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    for i in range(len(xs)):
        assert res[i] is not None
        for out in res[i]:
            assert sfda.sfda_workspace_status(out[3]) == 0
            for a, b in zip(out[:3], serial[i][:3]):
                assert torch.equal(a, b)


# ------------------------------------------------------------------------------------------------
# timing perturbation: a build whose roles pause at random must reproduce the plain build bit for bit
# ------------------------------------------------------------------------------------------------
def test_forward_results_do_not_depend_on_the_timing_of_the_roles():
    """The tensor-core forward hands tiles between four concurrently running roles through barriers.  No result
    may depend on how fast a role runs; a development build of the library (-DSFDA_WS_CHAOS) pauses every role for
    0.1 to 1.1 microseconds after one in eight barrier arrivals and completed waits.  A missing or misplaced
    synchronisation (a tile announced before it is complete, an accumulator read after the next product has
    started it from zero) shows as a bit difference between that build and the plain one.  Shapes: a ragged tail,
    time slices with hand-off between CTAs, the balanced partition, raw inputs, the two-level scan."""
    from paper_2607_11897_b200 import binding, build as cuda_build
    chaos = binding.load_library(cuda_build.build_variant("chaos", ["-DSFDA_WS_CHAOS"]))
    plain = binding.load()

    def with_lib(lib, fn):
        binding._LIB = lib
        try:
            return fn()
        finally:
            binding._LIB = plain

    def forward_case(B, T, H, s0, want_im, cut):
        cfg = workloads.CONFIGS[2].scaled(name="chaos", B=B, T=T, H=H, s0_std=s0, seed=900 + B + T + H)
        inp = workloads.forward_inputs(cfg)
        d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
        nws = sfda.sfda_workspace_bytes(B, T, H, 128, 128, 64, 1) if cut else 256

        def run():
            o = torch.empty(B, T, H, 128, device=DEV, dtype=torch.bfloat16)
            o_im = torch.empty_like(o) if want_im else None
            S_T = torch.empty(B, H, 128, 128, device=DEV)
            ws = torch.empty(nws, device=DEV, dtype=torch.uint8)
            sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, 64, ws)
            torch.cuda.synchronize()
            assert sfda.sfda_workspace_status(ws) == 0
            return [o, S_T] + ([o_im] if want_im else [])
        return run

    def fused_case(B, T, H):
        cfg = workloads.CONFIGS[2].scaled(name="chaosf", B=B, T=T, H=H, s0_std=0.02, seed=950 + T)
        raw = workloads.forward_raw_inputs(cfg)
        return lambda: [torch.from_numpy(x) for x in run_forward_fused(cfg, raw, PARAM)[:3]]

    def two_level_case(B, T, H, n):
        cfg = workloads.CONFIGS[3].scaled(name="chaos2", B=B, T=T, H=H, s0_std=0.3, seed=970)
        inp = workloads.forward_inputs(cfg)
        d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}

        def run():
            o = torch.empty(B, T, H, 128, device=DEV, dtype=torch.bfloat16)
            o_im = torch.empty_like(o)
            S_T = torch.empty(B, H, 128, 128, device=DEV)
            ws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(B, T, H, 128, 128, 64, 1, n), device=DEV,
                             dtype=torch.uint8)
            sfda.sfda_forward_two_level(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T,
                                        64, n, ws)
            torch.cuda.synchronize()
            return [o, o_im, S_T]
        return run

    cases = {
        "ragged tail, B = 4": forward_case(4, 1029, 8, 0.02, True, True),
        "time slices with hand-off (150 sequences of 64 chunks)": forward_case(1, 4096, 150, 0.02, True, True),
        "balanced partition (149 sequences of 4 chunks)": forward_case(1, 256, 149, 0.0, False, True),
        "uncut, one head": forward_case(2, 2048, 1, 0.02, True, False),
        "raw inputs": fused_case(3, 1029, 2),
        "raw inputs, time slices": fused_case(1, 2048, 150),
        "two-level scan": two_level_case(1, 4096, 3, 8),
    }
    for name, run in cases.items():
        want = with_lib(plain, run)
        for rep in range(3):
            got = with_lib(chaos, run)
            for x, y in zip(got, want):
                assert torch.equal(x, y), "%s: the build with random pauses differs from the plain build (launch %d)" % (name, rep)


# ------------------------------------------------------------------------------------------------
# a bounded device-side wait that runs out (no fault: the kernel gives up, reports, and ends)
# ------------------------------------------------------------------------------------------------
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """Two sequences of eight chunks, each cut into two time slices on four CTAs; the diagnostic launch writes the
    boundary states but never announces them, with the wait limit at 2^20 ticks of the SM clock (about half a
    millisecond).  The two CTAs that run second slices wait for their predecessors until the limit, give up, all
    their roles leave, tensor memory is freed and the kernel ends; the status word reads SFDA_ERR_TIMEOUT.  The first
    slices' outputs are still right, and an ordinary call on the same workspace afterwards is right everywhere."""
    cfg = workloads.CONFIGS[1].scaled(name="timeout", B=1, T=512, H=2, s0_std=0.1, seed=611)
    inp = workloads.forward_inputs(cfg)
    d = {k: (None if v is None else to_dev(v, cfg, k)) for k, v in inp.items()}
    o = torch.zeros(cfg.B, cfg.T, cfg.H, 128, device=DEV, dtype=torch.bfloat16)
    o_im = torch.zeros_like(o)
    S_T = torch.zeros(cfg.B, cfg.H, 128, 128, device=DEV)
    ws = torch.empty(sfda.sfda_workspace_bytes(cfg.B, cfg.T, cfg.H, 128, 128, 64, 1), device=DEV, dtype=torch.uint8)
    w_re, w_im, w_S = oracle_pairs(inp, all_pairs(cfg))
    sfda.sfda_forward_withheld_handoff(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T,
                                       64, 2, 1 << 20, ws)
    with pytest.raises(sfda.SfdaError) as e:
        sfda.sfda_workspace_status(ws)
    assert e.value.status == -7
    half = cfg.T // 2                                    # first slices: tokens 0 .. T/2 - 1 of both sequences
    got = np.stack([o.float().cpu().numpy()[0, :half, h] for h in range(cfg.H)])
    assert rel_err(got, w_re[:, :half]) <= TOL["bf16"]
    # argument checks of the diagnostic itself
    for slices, ticks, code in ((1, 1 << 20, -8), (2, 1 << 10, -8), (2, 1 << 30, -8), (3, 1 << 20, -2)):
        with pytest.raises(sfda.SfdaError) as e:
            sfda.sfda_forward_withheld_handoff(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im,
                                               S_T, 64, slices, ticks, ws)
        assert e.value.status == code
    # the context is intact: the ordinary call, on the very same workspace
    sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T, 64, ws)
    assert sfda.sfda_workspace_status(ws) == 0
    on, oin, Sn = o.float().cpu().numpy(), o_im.float().cpu().numpy(), S_T.cpu().numpy()
    assert rel_err(np.stack([on[0, :, h] for h in range(cfg.H)]), w_re) <= TOL["bf16"]
    assert rel_err(np.stack([oin[0, :, h] for h in range(cfg.H)]), w_im) <= TOL["bf16"]
    assert rel_err(np.stack([Sn[0, h] for h in range(cfg.H)]), w_S) <= TOL["bf16"]
