"""Seeded synthetic inputs shaped like the paper's two training set-ups.

Only input generation lives here: shapes, value distributions, padding / packing structure,
staleness draws and GRPO-style advantages.  None of the library's arithmetic (LM head,
log-softmax, interpolation, ratio, clip, reduction) is in this module, so both the CUDA path
and the CPU oracle can be fed from it without sharing method code.

The paper trains Qwen2.5-1.5B-Instruct on GSM8K (responses up to 1,024 tokens) and Qwen3-8B on
DAPO-Math-17k (responses up to 2,048 tokens) with mini-batches of at most 10,240 tokens
(Sec. 4.1).  Those datasets and weights are not needed for this path: its cost and numerics
depend only on shapes, mask density and dtype.  The generators below stand in for them with
the models' public head shapes (H = 1536 or 4096, V = 151,936), random-init weights and
random hidden states.

Small per-token / per-sequence arrays are drawn on the host with numpy's PCG64
(`default_rng(seed)`); the two large matrices (hidden, W) are drawn with a seeded
`torch.Generator` on the requested device.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 20251206 * 10

QWEN_VOCAB = 151936


@dataclass
class Workload:
    name: str
    dtype: str                    # "f32" or "bf16": storage type of hidden / W
    N: int                        # token rows (padded or packed)
    H: int
    V: int
    B: int                        # sequences
    cu_seqlens: np.ndarray        # int32 [B+1], row offsets of each sequence
    valid_len: np.ndarray         # int32 [B], response length of each sequence (<= row span)
    targets: np.ndarray           # int32 [N]
    versions: np.ndarray          # int32 [N]  behaviour-policy version per token
    versions_per_seq: np.ndarray  # int32 [B]
    current_version: int
    adv: np.ndarray               # fp32 [N]
    mask: np.ndarray              # uint8 [N]
    behav_noise: np.ndarray       # fp32 [N]: behaviour logp = min(current logp + noise, 0)
    clip_eps: float
    hidden: torch.Tensor | None = None   # [N,H] on `device`
    w: torch.Tensor | None = None        # [V,H] on `device`
    meta: dict = field(default_factory=dict)


# ------------------------------------------------------------------------------ pieces
def torch_dtype(dtype: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]


def lm_head_operands(n, h, v, dtype, seed, device="cpu"):
    """hidden ~ N(0,1) [n,h];  W ~ N(0, 1/h) [v,h]; rounded to `dtype` (RNE) after drawing in fp32."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    td = torch_dtype(dtype)
    hidden = torch.empty((n, h), dtype=td, device=device)
    w = torch.empty((v, h), dtype=td, device=device)
    slab = max(1, (1 << 26) // max(h, 1))          # bound the fp32 temporaries
    for lo in range(0, n, slab):
        hi = min(lo + slab, n)
        hidden[lo:hi] = torch.randn((hi - lo, h), generator=gen, device=device, dtype=torch.float32).to(td)
    scale = 1.0 / float(np.sqrt(h))
    for lo in range(0, v, slab):
        hi = min(lo + slab, v)
        w[lo:hi] = (torch.randn((hi - lo, h), generator=gen, device=device, dtype=torch.float32) * scale).to(td)
    return hidden, w


def peak_targets(hidden, w, rng, p_lo=0.3, p_hi=0.999, late_fraction=0.5):
    """Turns flat random rows into confident ones, the way an RL fine-tuning batch looks (sampled tokens
    mostly have high probability under the policy that is trained on them).

    Every row t gets its own target y_t (all distinct), half of them (late_fraction) in the last eighth of
    the vocabulary so that they fall into late column tiles and the last vocabulary split, and W[y_t] is
    moved along hidden[t] by the amount that lifts the target's logit to about
    ln V + 1/2 + logit(P_t) with P_t log-uniform in odds between p_lo and p_hi: the target probability
    then lands near P_t (the other V - 1 logits stay ~ N(0,1), whose log-sum-exp is ln V + 1/2).
    Modifies `w` in place (same dtype, rounded RNE) and returns the int32 targets [N] (numpy)."""
    n, h = hidden.shape
    v = w.shape[0]
    if n > v:
        raise ValueError("peak_targets needs at most V rows (targets are distinct)")
    n_late = min(int(n * late_fraction), max(v // 8, 1))
    late_pool = np.arange(v - max(v // 8, 1), v)
    late = rng.choice(late_pool, size=n_late, replace=False)
    rest_pool = np.setdiff1d(np.arange(v), late, assume_unique=False)
    rest = rng.choice(rest_pool, size=n - n_late, replace=False)
    targets = np.concatenate([late, rest]).astype(np.int32)
    rng.shuffle(targets)
    odds = np.exp(rng.uniform(np.log(p_lo / (1 - p_lo)), np.log(p_hi / (1 - p_hi)), size=n))
    lift = torch.from_numpy((np.log(v) + 0.5 + np.log(odds)).astype(np.float32)).to(hidden.device)
    hid = hidden.float()
    y = torch.from_numpy(targets.astype(np.int64)).to(hidden.device)
    base = (hid * w[y].float()).sum(dim=1)                       # the target's logit before the nudge
    step = ((lift - base) / (hid * hid).sum(dim=1).clamp_min(1e-6)).unsqueeze(1) * hid
    w[y] = (w[y].float() + step).to(w.dtype)
    return targets


def group_normalised_advantages(rewards, group_size, norm_eps=1e-6):
    """GRPO-style advantage, one per sequence: (R - mean_group) / (std_group + norm_eps)."""
    r = np.asarray(rewards, dtype=np.float64).reshape(-1, group_size)
    mean = r.mean(axis=1, keepdims=True)
    std = r.std(axis=1, keepdims=True)
    return ((r - mean) / (std + norm_eps)).reshape(-1).astype(np.float32)


def behav_logp_from(logp, noise):
    """Behaviour log-prob recipe shared by all configs: current + noise, never above 0."""
    return np.minimum(np.asarray(logp, dtype=np.float32) + np.asarray(noise, dtype=np.float32),
                      np.float32(0.0)).astype(np.float32)


def _broadcast(per_seq, cu):
    out = np.empty(int(cu[-1]), dtype=per_seq.dtype)
    for b in range(len(cu) - 1):
        out[cu[b]:cu[b + 1]] = per_seq[b]
    return out


def rl_batch(rng, *, n_prompts, group, row_len=None, len_lo, len_hi, packed, max_staleness=None,
             geometric_p=None, staleness_cap=None, reward_p=None, noise_std, mask_keep=None,
             current_version=32, v=QWEN_VOCAB):
    """Per-token and per-sequence arrays of one RL training batch.

    padded layout (packed=False): every sequence owns `row_len` rows; the first `valid_len`
    are response tokens, the rest is right padding with mask 0.
    packed layout (packed=True): sequences are concatenated (cu_seqlens), no padding rows.
    """
    b = n_prompts * group
    valid_len = rng.integers(len_lo, len_hi + 1, size=b).astype(np.int32)
    if packed:
        cu = np.concatenate([[0], np.cumsum(valid_len)]).astype(np.int64)
    else:
        cu = (np.arange(b + 1, dtype=np.int64) * row_len)
    n = int(cu[-1])
    if geometric_p is not None:
        d = np.minimum(rng.geometric(geometric_p, size=b) - 1, staleness_cap)
    else:
        d = rng.integers(0, max_staleness + 1, size=b)
    versions_per_seq = (current_version - d).astype(np.int32)
    if reward_p is None:
        adv_seq = rng.standard_normal(b).astype(np.float32)
    else:
        rewards = (rng.random(b) < reward_p).astype(np.float64)
        adv_seq = group_normalised_advantages(rewards, group)
    mask = np.zeros(n, dtype=np.uint8)
    for i in range(b):
        mask[cu[i]:cu[i] + valid_len[i]] = 1
    if mask_keep is not None:
        mask &= (rng.random(n) < mask_keep).astype(np.uint8)
    return dict(
        B=b, N=n, cu_seqlens=cu.astype(np.int32), valid_len=valid_len,
        targets=rng.integers(0, v, size=n).astype(np.int32),
        versions=_broadcast(versions_per_seq, cu), versions_per_seq=versions_per_seq,
        current_version=int(current_version), adv=_broadcast(adv_seq, cu), mask=mask,
        behav_noise=(rng.standard_normal(n) * noise_std).astype(np.float32),
    )


# ------------------------------------------------------------------------------ configs
_SHAPES = {
    # name: dtype, H, V, batch recipe
    "tiny": dict(dtype="f32", H=64, V=1000,
                 batch=dict(n_prompts=2, group=2, row_len=128, len_lo=128, len_hi=128, packed=False,
                            max_staleness=4, reward_p=None, noise_std=0.05, mask_keep=0.9,
                            current_version=8)),
    "1p5b": dict(dtype="bf16", H=1536, V=QWEN_VOCAB,
                 batch=dict(n_prompts=2, group=8, row_len=1024, len_lo=256, len_hi=1024, packed=False,
                            max_staleness=4, reward_p=0.5, noise_std=0.1)),
    "8b": dict(dtype="bf16", H=4096, V=QWEN_VOCAB,
               batch=dict(n_prompts=8, group=8, row_len=2048, len_lo=512, len_hi=2048, packed=False,
                          max_staleness=8, reward_p=0.3, noise_std=0.2)),
    "8b_packed": dict(dtype="bf16", H=4096, V=QWEN_VOCAB,
                      batch=dict(n_prompts=16, group=16, len_lo=512, len_hi=8192, packed=True,
                                 geometric_p=0.4, staleness_cap=16, reward_p=0.3, noise_std=0.3,
                                 mask_keep=0.95)),
}
_SEED_OFFSET = {"tiny": 0, "1p5b": 1, "8b": 2, "loss_sweep": 3, "8b_packed": 4}


def make_workload(name, device="cpu", *, H=None, V=None, dtype=None, with_operands=True,
                  seed=None, **batch_overrides) -> Workload:
    """Build one of the named workloads; H / V / dtype and any batch field (n_prompts, group,
    row_len, len_lo, len_hi, ...) may be overridden to make a shrunken copy with the same
    structure."""
    spec = _SHAPES[name]
    h = H or spec["H"]
    v = V or spec["V"]
    dt = dtype or spec["dtype"]
    seed = BASE_SEED + _SEED_OFFSET[name] if seed is None else seed
    rng = np.random.default_rng(seed)
    recipe = dict(spec["batch"])
    recipe.update(batch_overrides)
    batch = rl_batch(rng, v=v, **recipe)
    hidden = w = None
    if with_operands:
        hidden, w = lm_head_operands(batch["N"], h, v, dt, seed, device)
    return Workload(name=name, dtype=dt, H=h, V=v, clip_eps=0.2, hidden=hidden, w=w,
                    meta=dict(seed=seed, recipe=recipe), **batch)


def loss_sweep(n, seed=None, correlated=False):
    """Loss-only bandwidth workload: fp32 logp arrays, int32 per-token versions, fp32 advantage,
    uint8 mask.  Literal reading: current and behaviour logp both i.i.d. -Exponential(1).
    correlated=True instead draws behaviour = min(current + N(0,0.2), 0) so that most tokens sit
    inside the clip range."""
    seed = BASE_SEED + _SEED_OFFSET["loss_sweep"] if seed is None else seed
    rng = np.random.default_rng(seed)
    logp = (-rng.standard_exponential(n)).astype(np.float32)
    if correlated:
        behav = behav_logp_from(logp, rng.standard_normal(n).astype(np.float32) * np.float32(0.2))
    else:
        behav = (-rng.standard_exponential(n)).astype(np.float32)
    current_version = 32
    versions = (current_version - rng.integers(0, 9, size=n)).astype(np.int32)
    adv = rng.standard_normal(n).astype(np.float32)
    mask = (rng.random(n) < 0.9).astype(np.uint8)
    return dict(logp=logp, behav_logp=behav, versions=versions, current_version=current_version,
                adv=adv, mask=mask, clip_eps=0.2, N=n)
