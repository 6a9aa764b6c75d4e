"""Two streams at once.  The tensor-core launches keep their CTAs in step through counters in the library's device
image, one block of counters per launch; when the other stream's launch holds the SMs, a launch's CTAs start one by
one, its pacing waits run out and back off.  Pacing is advisory, so the results must be exactly those of the same
calls run alone (the kernels are deterministic), no status bit may be raised, and a sample of rows must match the
oracle."""
import numpy as np
import pytest
import torch

import paper_2512_06547_b200 as a3po
from oracle import a3po_oracle as orc
from paper_2512_06547_b200 import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda"


class Problem:
    def __init__(self, n, h, v, seed):
        self.n, self.h, self.v = n, h, v
        self.hidden, self.w = workloads.lm_head_operands(n, h, v, "bf16", seed, DEV)
        rng = np.random.default_rng(seed)
        self.targets_np = rng.integers(0, v, size=n).astype(np.int32)
        self.targets = torch.from_numpy(self.targets_np).to(DEV)
        g = (rng.standard_normal(n) / n).astype(np.float32)
        g[rng.random(n) < 0.25] = 0.0
        self.g_np = g
        self.g = torch.from_numpy(g).to(DEV)
        self.kept = a3po.new_workspace(a3po.a3po_kept_bytes(n, v))
        self.ws = a3po.new_workspace(max(a3po.a3po_token_logprobs_fwd_keep_workspace_bytes(n, h, v),
                                         a3po.a3po_token_logprobs_bwd_kept_workspace_bytes(n, h, v)))
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def run(self):
        """Forward keeping the softmax + backward from it, on the current stream; returns fresh outputs."""
        n, h, v = self.n, self.h, self.v
        logp, lse = torch.empty(n, device=DEV), torch.empty(n, device=DEV)
        gh = torch.empty_like(self.hidden)
        gw = torch.empty(v, h, dtype=torch.float32, device=DEV)
        a3po.a3po_token_logprobs_fwd_keep(self.hidden, self.w, self.targets, logp, lse, self.kept, self.ws,
                                          status=self.status)
        a3po.a3po_token_logprobs_bwd_kept(self.hidden, self.w, self.targets, lse, self.g, self.kept, gh, gw, self.ws,
                                          status=self.status)
        return logp, lse, gh, gw


def test_concurrent_streams_give_the_results_of_serial_calls():
    a = Problem(4096 + 77, 1024, 32768 + 24, 901)
    b = Problem(3000, 1536, 20000 + 8, 902)
    alone = [p.run() for p in (a, b)]
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(3):
        with torch.cuda.stream(s1):
            out_a = [a.run() for _ in range(2)][-1]
        with torch.cuda.stream(s2):
            out_b = [b.run() for _ in range(2)][-1]
        torch.cuda.synchronize()
        assert int(a.status.item()) == 0 and int(b.status.item()) == 0
        for got, want in ((out_a, alone[0]), (out_b, alone[1])):
            for x, y in zip(got, want):
                assert torch.equal(x, y)
    # and the values themselves: 48 sampled rows of each problem against the oracle
    for p, (logp, lse, gh, _) in ((a, out_a), (b, out_b)):
        rows = np.random.default_rng(5).choice(p.n, size=48, replace=False)
        hn = p.hidden[torch.from_numpy(rows).to(DEV)].double().cpu().numpy()
        wn = p.w.double().cpu().numpy()
        logp_ref, lse_ref = orc.token_logprobs_fwd(hn, wn, p.targets_np[rows])
        gh_ref, _ = orc.token_logprobs_bwd(hn, wn, p.targets_np[rows], p.g_np[rows].astype(np.float64))
        assert np.max(np.abs(logp.cpu().numpy()[rows] - logp_ref)) <= 2e-3
        assert np.max(np.abs(lse.cpu().numpy()[rows] - lse_ref)) <= 2e-3
        got = gh.double().cpu().numpy()[rows]
        assert np.linalg.norm(got - gh_ref) <= 1e-2 * np.linalg.norm(gh_ref)
