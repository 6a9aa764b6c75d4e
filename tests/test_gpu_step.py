"""GPU parity of the chained path (log-probs -> loss -> gradients) and of the host-buffer entry."""
import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from oracle import a3po_oracle as orc
from paper_2512_06547_b200 import workloads
from tests.helpers import GRAD_FRO_RTOL, LOGP_TOL_BF16, LOGP_TOL_F32, chained_loss_tol, rel_fro, row_rel_err, to_np64

pytestmark = pytest.mark.gpu
DEV = "cuda"


def oracle_step(wl, hidden, w):
    hn, wn = to_np64(hidden), to_np64(w)
    logp, lse = orc.token_logprobs_fwd(hn, wn, wl.targets)
    behav = workloads.behav_logp_from(logp, wl.behav_noise)
    # The GPU's loss stage consumes the GPU's own logp (|err| <= 2e-3 for bf16 inputs).  A token whose ratio
    # lies that close to a clip bound may legitimately land on the other branch, which flips its whole
    # gradient; such tokens are masked out of this chained comparison (the loss-only tests cover the bounds).
    terms = orc.loss_terms(logp, behav, wl.versions, wl.current_version, wl.adv, wl.mask, wl.clip_eps)
    wl.mask = (wl.mask.astype(bool) & (terms["margin"] > 1e-2 * terms["r"])).astype(np.uint8)
    logp = np.where(wl.mask != 0, logp, 0.0)
    args = (logp, behav, wl.versions, wl.current_version, wl.adv, wl.mask, wl.clip_eps)
    terms = orc.loss_terms(*args)
    loss, stats = orc.loss_fwd(*args)
    g = orc.loss_bwd(*args)
    gh, gw = orc.token_logprobs_bwd(hn, wn, wl.targets, g)
    ent = orc.token_entropy(hn, wn)
    return dict(logp=logp, lse=lse, behav=behav, loss=loss, stats=stats, g=g, gh=gh, gw=gw, terms=terms, ent=ent)


def check_against_oracle(tag, wl, ref, loss, n_valid, gh, gw, logp=None, ent=None):
    """Tolerances as stated for the path: logp 2e-3 (bf16 inputs) / 1e-5 max(1,|lse|) (fp32), gradients 1e-2
    relative Frobenius (1e-4 for fp32 inputs), the loss within what a log-prob error of that size can move it."""
    bf16 = wl.dtype == "bf16"
    logp_tol = LOGP_TOL_BF16 if bf16 else LOGP_TOL_F32 * 10       # |lse| ~ 7 on the fp32 config
    loss_tol = chained_loss_tol(ref["terms"], logp_tol)
    grad_tol = GRAD_FRO_RTOL if bf16 else 1e-4
    e_loss = abs(loss - ref["loss"])
    e_gh, e_gw = rel_fro(to_np64(gh), ref["gh"]), rel_fro(to_np64(gw), ref["gw"])
    live = ref["g"] != 0
    e_row = float(row_rel_err(to_np64(gh)[live], ref["gh"][live]).max()) if live.any() else 0.0
    print(f"[{tag}] |dL|={e_loss:.3e} (tol {loss_tol:.3e})  grad_hidden fro={e_gh:.3e} worst row={e_row:.3e}  "
          f"grad_w fro={e_gw:.3e}")
    assert e_loss <= loss_tol
    assert n_valid == ref["stats"]["n_valid"]
    assert e_gh <= grad_tol and e_gw <= grad_tol
    assert e_row <= (3 * GRAD_FRO_RTOL if bf16 else 1e-3)          # no single row is off, peaked ones included
    assert not to_np64(gh)[ref["g"] == 0].any()                    # masked and clipped rows: exactly zero
    if logp is not None:
        valid = wl.mask != 0
        assert np.max(np.abs(logp.cpu().numpy() - ref["logp"])[valid], initial=0.0) <= logp_tol
        assert not logp.cpu().numpy()[~valid].any()
    if ent is not None:
        valid = wl.mask != 0
        assert np.max(np.abs(ent.cpu().numpy() - ref["ent"])[valid], initial=0.0) <= 5e-3
        assert not ent.cpu().numpy()[~valid].any()


def run_host_step(wl, behav):
    dt = a3po.A3PO_F32 if wl.dtype == "f32" else a3po.A3PO_BF16
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_hidden = wl.hidden.cpu().pin_memory()
    stage = a3po.new_workspace(a3po.a3po_train_step_stage_bytes(wl.N, wl.H, dt))
    stage.fill_(0xFF)       # rows of hidden that are not copied (mask 0) read as NaN: nothing may depend on them
    ws = a3po.new_workspace(a3po.a3po_train_step_workspace_bytes(wl.N, wl.H, wl.V, dt))
    grad_w = torch.zeros((wl.V, wl.H), dtype=torch.float32, device=DEV)
    grad_hidden = torch.empty_like(wl.hidden)
    h_loss = torch.zeros(1).pin_memory()
    h_stats = torch.zeros(24, dtype=torch.uint8).pin_memory()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    copied = a3po.a3po_host_to_device_bytes()
    a3po.a3po_train_step_host(h_hidden, pin(wl.targets), pin(behav), pin(wl.versions), pin(wl.adv), pin(wl.mask),
                              wl.current_version, wl.clip_eps, wl.w, grad_w, grad_hidden, stage, ws, h_loss,
                              h_stats=h_stats, d_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # transfer accounting: the per-token arrays in full, of hidden at least the rows that take part, at most all
    copied = a3po.a3po_host_to_device_bytes() - copied
    row_bytes = wl.H * h_hidden.element_size()
    small = wl.N * (4 + 4 + 4 + 4 + 1)
    assert small + int((wl.mask != 0).sum()) * row_bytes <= copied <= small + wl.N * row_bytes
    if wl.dtype == "bf16" and wl.meta["recipe"].get("packed") is False:
        assert copied < small + wl.N * row_bytes          # right padding stays on the host
    return float(h_loss.item()), a3po.read_stats(h_stats), grad_hidden, grad_w


def make(name, kw, peaked):
    wl = workloads.make_workload(name, DEV, **kw)
    if peaked:   # confident rows, targets in late column tiles / the last vocabulary split
        wl.targets = workloads.peak_targets(wl.hidden, wl.w, np.random.default_rng(wl.meta["seed"] + 7))
    return wl


@pytest.mark.parametrize("name,kw,peaked", [
    ("tiny", {}, False),
    ("1p5b", dict(V=8192 + 24, n_prompts=1, group=4, row_len=160, len_lo=40, len_hi=160), False),
    ("1p5b", dict(V=8192 + 24, n_prompts=1, group=4, row_len=160, len_lo=40, len_hi=160), True),
    ("8b_packed", dict(V=4096 + 8, H=1024, n_prompts=2, group=3, len_lo=30, len_hi=300), False),
])
def test_chained_step_matches_oracle(name, kw, peaked):
    wl = make(name, kw, peaked)
    ref = oracle_step(wl, wl.hidden, wl.w)
    loss, stats, gh, gw = run_host_step(wl, ref["behav"])
    assert stats["n_clipped"] == ref["stats"]["n_clipped"]
    check_against_oracle(f"host step {name}{' peaked' if peaked else ''}", wl, ref, loss, stats["n_valid"], gh, gw)


def _device_step(wl, behav, ws_bytes, want_entropy=True):
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    n = wl.N
    out = dict(logp=torch.full((n,), 7.0, device=DEV), lse=torch.full((n,), 7.0, device=DEV),
               grad_logp=torch.full((n,), 7.0, device=DEV), loss=torch.zeros(1, device=DEV),
               grad_hidden=torch.full_like(wl.hidden, 7.0),
               grad_w=torch.full((wl.V, wl.H), 7.0, dtype=torch.float32, device=DEV), stats=a3po.new_stats(),
               entropy=torch.full((n,), 7.0, device=DEV) if want_entropy else None)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = a3po.new_workspace(ws_bytes)
    a3po.a3po_train_step(wl.hidden, wl.w, to_dev(wl.targets), to_dev(behav), to_dev(wl.versions), wl.current_version,
                         to_dev(wl.adv), to_dev(wl.mask), wl.clip_eps, out["logp"], out["lse"], out["grad_logp"],
                         out["loss"], out["grad_hidden"], out["grad_w"], ws, stats=out["stats"],
                         entropy=out["entropy"], status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out


@pytest.mark.parametrize("name,kw,peaked", [
    ("1p5b", dict(V=8192 + 24, n_prompts=2, group=4, row_len=200, len_lo=30, len_hi=200), False),
    ("1p5b", dict(V=8192 + 24, n_prompts=2, group=4, row_len=200, len_lo=30, len_hi=200), True),
    ("8b_packed", dict(V=2048 + 200, H=512, n_prompts=2, group=4, len_lo=20, len_hi=400), False),
    ("8b_packed", dict(V=2048 + 200, H=512, n_prompts=2, group=4, len_lo=20, len_hi=400), True),
])
def test_keeping_step_matches_recomputing_step_and_oracle(name, kw, peaked):
    """a3po_train_step with the recommended workspace (backward from the kept softmax) and with the minimum
    workspace (three calls, logits recomputed), each against the oracle; flat rows and peaked rows (target
    probability 0.3 .. 0.999, half of the targets in the last eighth of the vocabulary)."""
    wl = make(name, kw, peaked)
    ref = oracle_step(wl, wl.hidden, wl.w)          # also masks out tokens that sit on a clip bound
    dt = a3po.A3PO_BF16
    big = a3po.a3po_train_step_workspace_bytes(wl.N, wl.H, wl.V, dt)
    small = a3po.a3po_train_step_min_workspace_bytes(wl.N, wl.H, wl.V, dt)
    assert small < big
    outs = {"kept": _device_step(wl, ref["behav"], big), "recomputed": _device_step(wl, ref["behav"], small)}
    for tag, out in outs.items():
        check_against_oracle(f"{tag} {name}{' peaked' if peaked else ''}", wl, ref, float(out["loss"].item()),
                             a3po.read_stats(out["stats"])["n_valid"], out["grad_hidden"], out["grad_w"],
                             logp=out["logp"], ent=out["entropy"])
        g = out["grad_logp"].cpu().numpy()
        assert np.max(np.abs(g - ref["g"])) <= 1e-2 * np.max(np.abs(ref["g"])) + 1e-12
    # the two paths share the forward arithmetic up to the summation order of the softmax
    assert torch.allclose(outs["kept"]["logp"], outs["recomputed"]["logp"], atol=2e-4)
    assert rel_fro(to_np64(outs["kept"]["grad_w"]), to_np64(outs["recomputed"]["grad_w"])) <= GRAD_FRO_RTOL
    assert rel_fro(to_np64(outs["kept"]["grad_hidden"]), to_np64(outs["recomputed"]["grad_hidden"])) <= GRAD_FRO_RTOL


def test_keeping_step_in_several_row_chunks():
    """A batch long enough for a workspace that holds only part of it: the step runs the keeping path chunk by
    chunk (the loss accumulates over the chunks, grad_w is added to per chunk) and matches the one-chunk run
    and the oracle; grad_w accumulation into an existing buffer is checked on the way."""
    kw = dict(V=1024 + 40, H=256, n_prompts=3, group=4, row_len=640, len_lo=200, len_hi=640)
    wl = make("1p5b", kw, peaked=False)
    ref = oracle_step(wl, wl.hidden, wl.w)
    dt = a3po.A3PO_BF16
    big = a3po.a3po_train_step_workspace_bytes(wl.N, wl.H, wl.V, dt)
    vpad = (wl.V + 7) // 8 * 8
    per_row = 2 * vpad + 6 * wl.H + 2 * 4 * 64 + 5 * 4          # kept ratios, hidden_c + hs + ghc, split sums, row plan
    cap = (wl.N + 127) // 128 * 128
    assert cap >= 3 * 2048
    part = big - (cap - 2048 - 512) * per_row                    # room for chunks of a bit over 2048 rows
    one = _device_step(wl, ref["behav"], big)
    many = _device_step(wl, ref["behav"], part)
    for tag, out in (("one chunk", one), ("several chunks", many)):
        check_against_oracle(tag, wl, ref, float(out["loss"].item()), a3po.read_stats(out["stats"])["n_valid"],
                             out["grad_hidden"], out["grad_w"], logp=out["logp"], ent=out["entropy"])
    assert torch.equal(one["logp"], many["logp"]) and torch.equal(one["grad_logp"], many["grad_logp"])
    assert a3po.read_stats(one["stats"]) == a3po.read_stats(many["stats"])
    assert rel_fro(to_np64(many["grad_w"]), to_np64(one["grad_w"])) <= 1e-3
    launches0 = a3po.a3po_kernel_launch_count()
    _device_step(wl, ref["behav"], big)
    l_one = a3po.a3po_kernel_launch_count() - launches0
    _device_step(wl, ref["behav"], part)
    l_many = a3po.a3po_kernel_launch_count() - launches0 - l_one
    assert l_many > l_one                                         # it really ran in more than one chunk


@pytest.mark.parametrize("ws_kind", ["recommended", "min"])
def test_loss_scale_and_data_parallel_helpers(ws_kind):
    """loss_scale multiplies every gradient and leaves the loss alone (both workspace regimes); the data-parallel
    wrapper on one rank (M_global = M_local, weight 1) reproduces the plain step; a3po_mask_count and
    a3po_dp_loss_scale give M and M_r / M."""
    from paper_2512_06547_b200.data_parallel import gpu_data_parallel_step
    wl = make("1p5b", dict(V=2048 + 24, H=256, n_prompts=2, group=4, row_len=120, len_lo=30, len_hi=120), False)
    ref = oracle_step(wl, wl.hidden, wl.w)
    dt = a3po.A3PO_BF16
    size = a3po.a3po_train_step_workspace_bytes if ws_kind == "recommended" else a3po.a3po_train_step_min_workspace_bytes
    ws_bytes = size(wl.N, wl.H, wl.V, dt)
    plain = _device_step(wl, ref["behav"], ws_bytes)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    # counts and weights
    count = torch.zeros(1, dtype=torch.int64, device=DEV)
    a3po.a3po_mask_count(to_dev(wl.mask), count, a3po.new_workspace(a3po.a3po_mask_count_workspace_bytes()))
    assert int(count.item()) == int(wl.mask.sum())
    total = count * 4
    scale, weighted = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    a3po.a3po_dp_loss_scale(count, total, scale, loss_local=plain["loss"], weighted_loss=weighted)
    torch.cuda.synchronize()
    assert float(scale.item()) == 0.25 and float(weighted.item()) == pytest.approx(0.25 * float(plain["loss"].item()))
    # the step with that weight
    n = wl.N
    out = dict(logp=torch.empty(n, device=DEV), lse=torch.empty(n, device=DEV), grad_logp=torch.empty(n, device=DEV),
               loss=torch.zeros(1, device=DEV), grad_hidden=torch.empty_like(wl.hidden),
               grad_w=torch.empty((wl.V, wl.H), dtype=torch.float32, device=DEV))
    ws = a3po.new_workspace(ws_bytes)
    a3po.a3po_train_step(wl.hidden, wl.w, to_dev(wl.targets), to_dev(ref["behav"]), to_dev(wl.versions),
                         wl.current_version, to_dev(wl.adv), to_dev(wl.mask), wl.clip_eps, out["logp"], out["lse"],
                         out["grad_logp"], out["loss"], out["grad_hidden"], out["grad_w"], ws, loss_scale=scale)
    torch.cuda.synchronize()
    assert float(out["loss"].item()) == float(plain["loss"].item())
    assert torch.allclose(out["grad_logp"], 0.25 * plain["grad_logp"], rtol=1e-6, atol=0)
    assert rel_fro(to_np64(out["grad_w"]), 0.25 * to_np64(plain["grad_w"])) <= 5e-3        # bf16 roundings differ
    assert rel_fro(to_np64(out["grad_hidden"]), 0.25 * to_np64(plain["grad_hidden"])) <= 5e-3
    # the wrapper on a single rank
    batch = dict(hidden=wl.hidden, w=wl.w, targets=to_dev(wl.targets), behav_logp=to_dev(ref["behav"]),
                 versions=to_dev(wl.versions), current_version=wl.current_version, adv=to_dev(wl.adv),
                 mask=to_dev(wl.mask), clip_eps=wl.clip_eps, ws=ws, **out)
    res = gpu_data_parallel_step()(batch)
    torch.cuda.synchronize()
    assert float(res["scale"].item()) == 1.0 and int(res["m_global"].item()) == int(wl.mask.sum())
    assert float(res["loss"].item()) == pytest.approx(float(plain["loss"].item()), rel=1e-6)
    assert torch.equal(res["grad_w"], plain["grad_w"]) and torch.equal(res["grad_logp"], plain["grad_logp"])


def test_step_replays_from_a_cuda_graph():
    """The whole step is a fixed sequence of launches on one stream (row counts stay on the device), so it can be
    captured once and replayed: same bits as the eager call, for new input values in the same buffers too."""
    wl = make("1p5b", dict(V=8192 + 24, n_prompts=2, group=4, row_len=200, len_lo=30, len_hi=200), True)
    ref = oracle_step(wl, wl.hidden, wl.w)
    dt = a3po.A3PO_BF16
    ws_bytes = a3po.a3po_train_step_workspace_bytes(wl.N, wl.H, wl.V, dt)
    eager = _device_step(wl, ref["behav"], ws_bytes)              # also the uncaptured first call on this device
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    n = wl.N
    targets, behav, versions, adv, mask = (to_dev(x) for x in (wl.targets, ref["behav"], wl.versions, wl.adv, wl.mask))
    out = dict(logp=torch.empty(n, device=DEV), lse=torch.empty(n, device=DEV), grad_logp=torch.empty(n, device=DEV),
               loss=torch.zeros(1, device=DEV), grad_hidden=torch.empty_like(wl.hidden),
               grad_w=torch.empty((wl.V, wl.H), dtype=torch.float32, device=DEV), entropy=torch.empty(n, device=DEV))
    stats = a3po.new_stats()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = a3po.new_workspace(ws_bytes)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        a3po.a3po_train_step(wl.hidden, wl.w, targets, behav, versions, wl.current_version, adv, mask, wl.clip_eps,
                             out["logp"], out["lse"], out["grad_logp"], out["loss"], out["grad_hidden"], out["grad_w"],
                             ws, stats=stats, entropy=out["entropy"], status=status)
    for _ in range(2):
        for t in out.values():
            t.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for k, t in out.items():
            assert torch.equal(t, eager[k]), k
    # other inputs in the same buffers: half of the tokens masked out, the replay follows the device-side counts
    mask2 = wl.mask.copy()
    mask2[::2] = 0
    mask.copy_(to_dev(mask2))
    graph.replay()
    torch.cuda.synchronize()
    wl.mask = mask2
    eager2 = _device_step(wl, ref["behav"], ws_bytes)
    for k, t in out.items():
        assert torch.equal(t, eager2[k]), k
