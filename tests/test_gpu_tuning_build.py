"""The kernel variants that only a tuning build (-DA3PO_TUNING) can select stay correct: the forward on CTA pairs
(tcgen05 cta_group::2), the gradient contractions on 128 x 256 tiles, and the persistent CTAs unpaced or paced at
every k-block.  Each variant runs in a child process,
because the switches are environment variables read by the tuning library."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_2512_06547_b200 import build as a3po_build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    import numpy as np, torch
    sys.path.insert(0, {root!r})
    from paper_2512_06547_b200 import binding
    binding.LIB_PATH = {lib!r}
    import paper_2512_06547_b200 as a3po
    from oracle import a3po_oracle as orc
    from paper_2512_06547_b200 import workloads
    dev = "cuda"
    for n, h, v in ((515, 1536, 4096 + 37), (257, 72, 1000), (700, 512, 5000 + 24)):
        hidden, w = workloads.lm_head_operands(n, h, v, "bf16", 400 + n, dev)
        rng = np.random.default_rng(n)
        t_np = workloads.peak_targets(hidden, w, rng) if n < v else rng.integers(0, v, size=n).astype(np.int32)
        targets = torch.from_numpy(t_np).to(dev)
        g_np = (rng.standard_normal(n) / n).astype(np.float32); g_np[rng.random(n) < 0.2] = 0
        g = torch.from_numpy(g_np).to(dev)
        hn, wn = hidden.double().cpu().numpy(), w.double().cpu().numpy()
        logp_ref, lse_ref = orc.token_logprobs_fwd(hn, wn, t_np)
        gh_ref, gw_ref = orc.token_logprobs_bwd(hn, wn, t_np, g_np.astype(np.float64))
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        # plain pair
        ws = a3po.new_workspace(max(a3po.a3po_token_logprobs_workspace_bytes(n, h, v, 1, 0), a3po.a3po_token_logprobs_workspace_bytes(n, h, v, 1, 1)))
        logp, lse = torch.empty(n, device=dev), torch.empty(n, device=dev)
        gh = torch.empty_like(hidden); gw = torch.empty(v, h, device=dev)
        a3po.a3po_token_logprobs_fwd(hidden, w, targets, logp, lse, ws, status=status)
        a3po.a3po_token_logprobs_bwd(hidden, w, targets, lse, g, gh, gw, ws, status=status)
        # keeping pair
        kept = a3po.new_workspace(a3po.a3po_kept_bytes(n, v))
        ws2 = a3po.new_workspace(max(a3po.a3po_token_logprobs_fwd_keep_workspace_bytes(n, h, v), a3po.a3po_token_logprobs_bwd_kept_workspace_bytes(n, h, v)))
        k_logp, k_lse = torch.empty(n, device=dev), torch.empty(n, device=dev)
        k_gh = torch.empty_like(hidden); k_gw = torch.empty(v, h, device=dev)
        a3po.a3po_token_logprobs_fwd_keep(hidden, w, targets, k_logp, k_lse, kept, ws2, status=status)
        a3po.a3po_token_logprobs_bwd_kept(hidden, w, targets, k_lse, g, kept, k_gh, k_gw, ws2, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        fro = lambda a, b: float(np.linalg.norm(a.double().cpu().numpy() - b) / np.linalg.norm(b))
        for lp, ls, a, b in ((logp, lse, gh, gw), (k_logp, k_lse, k_gh, k_gw)):
            assert np.max(np.abs(lp.cpu().numpy() - logp_ref)) <= 2e-3 and np.max(np.abs(ls.cpu().numpy() - lse_ref)) <= 2e-3
            assert fro(a, gh_ref) <= 1e-2 and fro(b, gw_ref) <= 1e-2
    print("variant ok")
""")


@pytest.mark.parametrize("env", [{"A3PO_FWD_PAIR": "1"}, {"A3PO_GRAD_MT": "1"}, {"A3PO_GRAD_MT": "2", "A3PO_FWD_PAIR": "1"},
                                 {"A3PO_PACE_OFF": "1"}, {"A3PO_PACE_PERIOD": "1", "A3PO_PACE_SLACK": "1"}])
def test_tuning_variants_match_the_oracle(env):
    lib = a3po_build.build(tuning=True)
    child_env = dict(os.environ, **env)
    res = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT, lib=lib)], env=child_env, capture_output=True,
                         text=True, timeout=600)
    assert res.returncode == 0 and "variant ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]
