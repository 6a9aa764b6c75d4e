"""Out-of-bounds evidence without a memory checker: every output and workspace of an ABI call sits inside a larger
allocation whose margins ("guard bands", 4 KiB before and after, the trailing one starting at the first byte past
the buffer) are filled with a pattern; after the call the bands must be untouched.  Ragged shapes (row, column
and K tails, shapes the tensor-core path rejects), workspaces of exactly the minimum and exactly the recommended
size.  Reads cannot be caught this way; writes outside a buffer can."""
import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from paper_2512_06547_b200 import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda"
BAND = 4096
PATTERN = 0xC3


class Guarded:
    """Allocates typed buffers with guard bands and checks all of them at once."""

    def __init__(self):
        self.items = []

    def new(self, name, shape, dtype, fill=None):
        numel = int(np.prod(shape)) if len(shape) else 1
        nbytes = numel * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((BAND + nbytes + BAND,), PATTERN, dtype=torch.uint8, device=DEV)
        inner = raw[BAND:BAND + nbytes].view(dtype).view(*shape) if nbytes else raw[BAND:BAND].view(dtype)
        assert raw.data_ptr() % 256 == 0          # so that the interior is 256-byte aligned as well
        if fill is not None and nbytes:
            inner.fill_(fill)
        self.items.append((name, raw, nbytes))
        return inner

    def check(self, where):
        torch.cuda.synchronize()
        for name, raw, nbytes in self.items:
            head, tail = raw[:BAND], raw[BAND + nbytes:]
            assert bool((head == PATTERN).all()), f"{where}: bytes before `{name}` were written"
            assert bool((tail == PATTERN).all()), f"{where}: bytes after `{name}` were written"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("n,h,v,dtype", [(131, 256, 777, "bf16"), (257, 72, 1000, "bf16"), (33, 12, 50, "bf16"),
                                         (300, 1536, 2048 + 40, "bf16"), (65, 40, 129, "f32")])
@pytest.mark.parametrize("ws_kind", ["min", "recommended"])
def test_lm_head_calls_stay_inside_their_buffers(n, h, v, dtype, ws_kind):
    hidden, w = workloads.lm_head_operands(n, h, v, dtype, 700 + n, DEV)
    rng = np.random.default_rng(n)
    targets = _dev(rng.integers(0, v, size=n).astype(np.int32))
    mask = _dev((rng.random(n) < 0.8).astype(np.uint8))
    g_np = (rng.standard_normal(n) / n).astype(np.float32)
    g_np[rng.random(n) < 0.3] = 0.0
    g = _dev(g_np) * mask
    dt = a3po.A3PO_F32 if dtype == "f32" else a3po.A3PO_BF16
    size = (a3po.a3po_token_logprobs_min_workspace_bytes if ws_kind == "min"
            else a3po.a3po_token_logprobs_workspace_bytes)
    G = Guarded()
    logp, lse, ent = (G.new(k, (n,), torch.float32, 9.0) for k in ("logp", "lse", "entropy"))
    status = G.new("status", (1,), torch.int32, 0)
    ws_f = G.new("ws_fwd", (size(n, h, v, dt, 0),), torch.uint8)
    a3po.a3po_token_logprobs_fwd(hidden, w, targets, logp, lse, ws_f, row_mask=mask, entropy=ent, status=status)
    G.check("token_logprobs_fwd")
    gh = G.new("grad_hidden", (n, h), hidden.dtype, 3.0)
    gw = G.new("grad_w", (v, h), torch.float32, 3.0)
    ws_b = G.new("ws_bwd", (size(n, h, v, dt, 1),), torch.uint8)
    a3po.a3po_token_logprobs_bwd(hidden, w, targets, lse, g, gh, gw, ws_b, status=status)
    a3po.a3po_token_logprobs_bwd(hidden, w, targets, lse, g, gh, gw, ws_b, accumulate_grad_w=True, status=status)
    G.check("token_logprobs_bwd")
    assert int(status.item()) == 0 and torch.isfinite(gw).all()


@pytest.mark.parametrize("n,h,v", [(131, 256, 777), (257, 72, 1000), (300, 1536, 2048 + 40), (1, 8, 9)])
def test_keep_pair_stays_inside_its_buffers(n, h, v):
    hidden, w = workloads.lm_head_operands(n, h, v, "bf16", 800 + n, DEV)
    rng = np.random.default_rng(n + 1)
    targets = _dev(rng.integers(0, v, size=n).astype(np.int32))
    mask = _dev((rng.random(n) < 0.8).astype(np.uint8))
    g = _dev((rng.standard_normal(n) / n).astype(np.float32)) * mask
    G = Guarded()
    logp, lse, ent = (G.new(k, (n,), torch.float32, 9.0) for k in ("logp", "lse", "entropy"))
    status = G.new("status", (1,), torch.int32, 0)
    kept = G.new("kept", (a3po.a3po_kept_bytes(n, v),), torch.uint8)
    ws_f = G.new("ws_fwd_keep", (a3po.a3po_token_logprobs_fwd_keep_workspace_bytes(n, h, v),), torch.uint8)
    a3po.a3po_token_logprobs_fwd_keep(hidden, w, targets, logp, lse, kept, ws_f, row_mask=mask, entropy=ent,
                                      status=status)
    G.check("token_logprobs_fwd_keep")
    gh = G.new("grad_hidden", (n, h), torch.bfloat16, 3.0)
    gw = G.new("grad_w", (v, h), torch.float32, 3.0)
    ws_b = G.new("ws_bwd_kept", (a3po.a3po_token_logprobs_bwd_kept_workspace_bytes(n, h, v),), torch.uint8)
    a3po.a3po_token_logprobs_bwd_kept(hidden, w, targets, lse, g, kept, gh, gw, ws_b, status=status)
    G.check("token_logprobs_bwd_kept")
    assert int(status.item()) == 0 and torch.isfinite(gw).all()


@pytest.mark.parametrize("n", [0, 1, 5, 1023, 100_003])
def test_loss_calls_stay_inside_their_buffers(n):
    inp = workloads.loss_sweep(n, seed=40 + n % 13, correlated=True)
    logp, behav, versions, adv, mask = (_dev(inp[k]) for k in ("logp", "behav_logp", "versions", "adv", "mask"))
    common = (logp, behav, versions, inp["current_version"], adv, mask, inp["clip_eps"])
    G = Guarded()
    loss = G.new("loss", (1,), torch.float32, 5.0)
    stats = G.new("stats", (24,), torch.uint8, 0)
    grad = G.new("grad_logp", (n,), torch.float32, 5.0)
    ws = G.new("ws", (a3po.a3po_loss_workspace_bytes(n),), torch.uint8)
    a3po.a3po_loss_fwd(*common, loss, ws, stats=stats)
    G.check("loss_fwd")
    a3po.a3po_loss_bwd(*common, grad, ws, fwd_stats=stats)
    a3po.a3po_loss_bwd(*common, grad, ws, detach_prox=False)
    G.check("loss_bwd")
    a3po.a3po_loss_fwd_bwd(*common, loss, grad, ws, stats=stats)
    G.check("loss_fwd_bwd")
    a3po.a3po_decoupled_loss_fwd_bwd(logp, behav, behav, adv, mask, inp["clip_eps"], loss, ws, grad_logp=grad, stats=stats)
    G.check("decoupled_loss_fwd_bwd")
    if n and n <= (1 << 20):
        a3po.a3po_loss_fwd_static(*common, loss, stats=stats)
        G.check("loss_fwd_static")


@pytest.mark.parametrize("name,kw", [
    ("tiny", {}),
    ("1p5b", dict(V=4096 + 24, n_prompts=1, group=4, row_len=150, len_lo=40, len_hi=150)),
    ("8b_packed", dict(V=2048 + 200, H=512, n_prompts=2, group=3, len_lo=20, len_hi=333)),
])
@pytest.mark.parametrize("ws_kind", ["min", "recommended"])
def test_train_step_stays_inside_its_buffers(name, kw, ws_kind):
    wl = workloads.make_workload(name, DEV, **kw)
    n, h, v = wl.N, wl.H, wl.V
    dt = a3po.A3PO_F32 if wl.dtype == "f32" else a3po.A3PO_BF16
    size = a3po.a3po_train_step_min_workspace_bytes if ws_kind == "min" else a3po.a3po_train_step_workspace_bytes
    behav = workloads.behav_logp_from(np.full(n, -7.0, dtype=np.float32), wl.behav_noise)
    G = Guarded()
    logp, lse, ent, grad_logp = (G.new(k, (n,), torch.float32, 9.0) for k in ("logp", "lse", "entropy", "grad_logp"))
    loss = G.new("loss", (1,), torch.float32, 5.0)
    stats = G.new("stats", (24,), torch.uint8, 0)
    status = G.new("status", (1,), torch.int32, 0)
    gh = G.new("grad_hidden", (n, h), wl.hidden.dtype, 3.0)
    gw = G.new("grad_w", (v, h), torch.float32, 3.0)
    ws = G.new("ws", (size(n, h, v, dt),), torch.uint8)
    a3po.a3po_train_step(wl.hidden, wl.w, _dev(wl.targets), _dev(behav), _dev(wl.versions), wl.current_version,
                         _dev(wl.adv), _dev(wl.mask), wl.clip_eps, logp, lse, grad_logp, loss, gh, gw, ws, stats=stats,
                         entropy=ent, status=status)
    G.check(f"train_step ({ws_kind} workspace)")
    assert int(status.item()) == 0 and torch.isfinite(gw).all() and torch.isfinite(loss).all()
    assert a3po.read_stats(stats)["n_valid"] == int(wl.mask.sum())
