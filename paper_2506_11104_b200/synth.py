"""Seeded synthetic inputs for the DAM prefill path.

This module only draws numbers and plants structure in Q and K.  It holds none of the
method's arithmetic (no softmax, no threshold, no pattern matching, no attention), so it
can feed both the CUDA library and the CPU checker with the very same arrays.

What is planted mirrors what the paper observes in real attention maps (Sec. 4.1 and
Appendix A): a sink column at token 0, a local diagonal band, and a few vertical stripes.
Each query head of a GQA group gets its own seeded mix on top of shared K/V:

* noise: Q, K, V ~ N(0, 1); rotary position embedding (theta 500000, rotate-half pairing,
  position = index inside the sequence) is applied to Q and K; the planted coordinates are
  then overwritten, so the structure below is exact;
* band: K carries ``n_harm`` unit harmonics (cos, sin)(2*pi*k*t / P), P = 2 * PCL; the query
  head carries Fejer weights over its first ``band_m`` harmonics, so the logit is
  ``amp * F_m(i - j)`` with F_m the Fejer kernel (peak 1 at 0, first zero at P / band_m,
  non-negative side lobes below 5 %).  Token 0's key and the stripe keys carry no band code;
* sink: one coordinate; every query of a head with a sink has it set, and so has key 0;
* stripes: one coordinate per query head of the group; the stripe keys of head h have it set
  in coordinate (h mod group), and so have all queries of head h.

All three peak logits equal ``amp``: a softmax is winner-take-all, so components must tie
to survive together.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch


@dataclass
class HeadPlan:
    sink: bool = True
    band_m: int = 0                 # 0 = no band; else number of Fejer harmonics (small = wide band)
    stripes: List[int] = field(default_factory=list)   # key positions inside the sequence


@dataclass
class Workload:
    name: str
    Q: torch.Tensor                 # [T, Hq, d]
    K: torch.Tensor                 # [T, Hkv, d]
    V: torch.Tensor                 # [T, Hkv, d]
    cu_seqlens: List[int]
    pcl_max: int
    tau: float
    mu: float
    lam: float = 0.5
    eps: float = 1e-8
    plans: Optional[List[List[HeadPlan]]] = None   # [seq][head]

    @property
    def num_q_heads(self):
        return self.Q.shape[1]

    @property
    def num_kv_heads(self):
        return self.K.shape[1]

    @property
    def head_dim(self):
        return self.Q.shape[2]

    @property
    def max_seqlen(self):
        return max(b - a for a, b in zip(self.cu_seqlens[:-1], self.cu_seqlens[1:]))


def _gen(seed_words: Sequence[int], device) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for w in seed_words:
        s = (s * 6364136223846793005 + 1442695040888963407 + int(w)) % (1 << 63)
    g.manual_seed(s)
    return g


def _rope(x: torch.Tensor, theta: float) -> torch.Tensor:
    """Rotate-half rotary embedding on x [S, H, d]; position = row index."""
    S, H, d = x.shape
    half = d // 2
    inv = theta ** (-torch.arange(0, half, device=x.device, dtype=torch.float32) / half)
    ang = torch.arange(S, device=x.device, dtype=torch.float32)[:, None] * inv[None, :]
    c, s = ang.cos()[:, None, :], ang.sin()[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * c - x2 * s, x1 * s + x2 * c], dim=-1)


def layout(d: int, group: int):
    """Coordinates reserved for planted structure: (n_harm, band dims, sink dim, first stripe dim)."""
    n_harm = 40 if d >= 128 else max(4, (d // 2 - group - 1) // 2)
    band = 2 * n_harm
    return n_harm, band, band, band + 1


def make_sequence(S: int, Hq: int, Hkv: int, d: int, pcl: int, plans: Sequence[HeadPlan], amp: float,
                  seed_words: Sequence[int], device="cpu", rope_theta: Optional[float] = 500000.0):
    """One sequence: float32 Q [S, Hq, d], K, V [S, Hkv, d]."""
    g = Hq // Hkv
    n_harm, band_dims, sink_dim, stripe0 = layout(d, g)
    n_res = stripe0 + g
    assert n_res <= d
    gen = _gen(seed_words, device)
    Q = torch.randn(S, Hq, d, generator=gen, device=device, dtype=torch.float32)
    K = torch.randn(S, Hkv, d, generator=gen, device=device, dtype=torch.float32)
    V = torch.randn(S, Hkv, d, generator=gen, device=device, dtype=torch.float32)
    if rope_theta:
        Q = _rope(Q, rope_theta)
        K = _rope(K, rope_theta)
    Q[:, :, :n_res] = 0.0
    K[:, :, :n_res] = 0.0

    rt = math.sqrt(amp * math.sqrt(d))        # q and k each carry sqrt(amp * sqrt(d)); product / sqrt(d) = amp
    pos = torch.arange(S, device=device, dtype=torch.float64)
    P = 2.0 * pcl
    kk = torch.arange(n_harm, device=device, dtype=torch.float64)
    ang = 2.0 * math.pi * pos[:, None] * kk[None, :] / P          # [S, n_harm]
    cs = torch.stack([ang.cos(), ang.sin()], dim=-1).reshape(S, band_dims).to(torch.float32)
    K[:, :, :band_dims] = cs[:, None, :]
    if S > 0:
        K[0, :, :band_dims] = 0.0
        K[0, :, sink_dim] = rt
    for h, plan in enumerate(plans):
        if plan.band_m > 0:
            m = min(plan.band_m, n_harm)
            # Fejer weights: F_m(x) = 1/m + (2/m) * sum_{k=1}^{m-1} (1 - k/m) cos(k x); F_m(0) = 1
            w = torch.zeros(n_harm, dtype=torch.float64, device=device)
            w[0] = 1.0 / m
            if m > 1:
                k = torch.arange(1, m, device=device, dtype=torch.float64)
                w[1:m] = (2.0 / m) * (1.0 - k / m)
            coef = (amp * math.sqrt(d)) * w                     # logit = sum_k coef_k cos(k x) / sqrt(d)
            Q[:, h, :band_dims] = (cs.to(torch.float64).reshape(S, n_harm, 2) * coef[None, :, None]) \
                .reshape(S, band_dims).to(torch.float32)
        if plan.sink:
            Q[:, h, sink_dim] = rt
        if plan.stripes:
            sd = stripe0 + (h % g)
            Q[:, h, sd] = rt
            idx = torch.tensor([p for p in plan.stripes if 0 < p < S], device=device, dtype=torch.long)
            if idx.numel():
                K[idx, h // g, sd] = rt
                K[idx, h // g, :band_dims] = 0.0     # a stripe key carries no band code (nor does the sink key)
    return Q, K, V


def _draw_plans(Hq: int, pcl: int, seed_words, band_m_choices: Sequence[int], max_stripes: int,
                sink_prob: float = 1.0, stripe_span: float = 0.5, stripe_skew: float = 1.0) -> List[HeadPlan]:
    gen = _gen(list(seed_words) + [7777], "cpu")
    plans = []
    for h in range(Hq):
        u = torch.rand(4, generator=gen)
        bm = band_m_choices[int(u[0] * len(band_m_choices)) % len(band_m_choices)]
        ns = int(float(u[1]) ** stripe_skew * (max_stripes + 1)) % (max_stripes + 1)   # skew > 1: mostly few, sometimes many
        # stripes inside the first `stripe_span` of the window (0.5: the first half)
        pos = torch.randperm(max(1, int(pcl * stripe_span) - 1), generator=gen)[:ns] + 1
        plans.append(HeadPlan(sink=bool(u[2] < sink_prob), band_m=int(bm), stripes=sorted(int(p) for p in pos)))
    return plans


def _pack(name, seqs, cu, pcl, tau, mu, dtype, plans) -> Workload:
    Q = torch.cat([s[0] for s in seqs], dim=0).to(dtype).contiguous()
    K = torch.cat([s[1] for s in seqs], dim=0).to(dtype).contiguous()
    V = torch.cat([s[2] for s in seqs], dim=0).to(dtype).contiguous()
    return Workload(name=name, Q=Q, K=K, V=V, cu_seqlens=list(cu), pcl_max=pcl, tau=tau, mu=mu, plans=plans)


# Mask-rule parameters per configuration.  tau is the paper's sparsity knob (Sec. 4.2.3); the paper's
# 0.3 keeps at most 44 keys per row, too few for the 64-512 wide bands these workloads ask for.
CONFIG_RULE = {
    0: dict(tau=0.10, mu=0.8, amp=8.0),
    1: dict(tau=0.05, mu=0.8, amp=10.0),
    2: dict(tau=0.05, mu=0.8, amp=10.0),
    3: dict(tau=0.05, mu=0.8, amp=10.0),
    4: dict(tau=0.05, mu=0.8, amp=10.0),
}


def config0(device="cpu") -> Workload:
    """Tiny case: 1 layer, 2 heads (MHA), d 64, S 512, PCL 128, fp32, seed 0.
    Head 0: sink + narrow local band.  Head 1: four stripes at seeded positions (< 64)."""
    S, H, d, pcl = 512, 2, 64, 128
    r = CONFIG_RULE[0]
    gen = _gen([0, 0, 99], "cpu")
    stripes = sorted(int(p) + 1 for p in torch.randperm(62, generator=gen)[:4])
    plans = [HeadPlan(sink=True, band_m=4, stripes=[]), HeadPlan(sink=False, band_m=0, stripes=stripes)]
    seq = make_sequence(S, H, H, d, pcl, plans, r["amp"], [0, 0, 0, 0], device)
    return _pack("C0 tiny fp32", [seq], [0, S], pcl, r["tau"], r["mu"], torch.float32, [plans])


def llama_layer(S: int, pcl: int, cfg: int, layer: int = 0, device="cpu", band_m_choices=(0, 2, 3, 4, 6, 8, 12, 16, 24, 40),
                max_stripes: int = 16, dtype=torch.bfloat16, name: Optional[str] = None, sink_prob: float = 1.0,
                stripe_span: float = 0.5, stripe_skew: float = 1.0, lone_stripe_heads: Sequence[int] = ()) -> Workload:
    """Llama-3-8B-shaped layer: 32 query heads, 8 KV heads, d 128, one sequence of S tokens.
    `lone_stripe_heads`: heads that attend to their first one or two stripe keys only (the sparsest masks)."""
    Hq, Hkv, d = 32, 8, 128
    r = CONFIG_RULE[cfg]
    plans = _draw_plans(Hq, pcl, [0, cfg, layer, 0], band_m_choices, max_stripes, sink_prob, stripe_span, stripe_skew)
    for k, h in enumerate(lone_stripe_heads):
        keys = plans[h].stripes[:1 + k % 2] or [pcl // 3 + 7 * k]
        plans[h] = HeadPlan(sink=False, band_m=0, stripes=keys)
    seq = make_sequence(S, Hq, Hkv, d, pcl, plans, r["amp"], [0, cfg, layer, 0], device)
    return _pack(name or f"C{cfg} layer {layer} S={S} PCL={pcl}", [seq], [0, S], pcl, r["tau"], r["mu"], dtype, [plans])


def config1(device="cpu") -> Workload:
    """Heads from a lone stripe or sink (a few per cent of the causal tiles) to the widest band the threshold
    keeps plus stripes all over the window (about 40 %)."""
    return llama_layer(8192, 1024, 1, 0, device, band_m_choices=(0, 0, 2, 2, 3, 4, 6, 8, 12, 16, 24, 40), max_stripes=32,
                       sink_prob=0.8, stripe_span=0.95, stripe_skew=3.0, lone_stripe_heads=(3, 14, 25))


def config2_layer(layer: int, device="cpu", S: int = 32768, pcl: int = 2048) -> Workload:
    """One layer of the 32-layer stack; the band/stripe mix is re-drawn per layer."""
    choices = [(0, 2, 2, 3, 4, 6), (0, 8, 12, 16, 24, 40), (2, 2, 4, 8, 16, 40), (0, 0, 24, 40)][layer % 4]
    return llama_layer(S, pcl, 2, layer, device, band_m_choices=choices, max_stripes=(8, 40, 64, 2)[layer % 4],
                       sink_prob=0.85, stripe_span=0.95, stripe_skew=(1.0, 1.0, 0.5, 1.0)[layer % 4])


def config3(device="cpu", S: int = 131072, pcl: int = 4096) -> Workload:
    return llama_layer(S, pcl, 3, 0, device, band_m_choices=(12, 16, 24), max_stripes=8)


def config4(device="cpu", lengths=(4096, 16384, 32768, 65536), pcl: int = 1024) -> Workload:
    """Ragged batch packed with cu_seqlens; every sequence has its own per-head plans."""
    Hq, Hkv, d = 32, 8, 128
    r = CONFIG_RULE[4]
    seqs, plans, cu = [], [], [0]
    for b, S in enumerate(lengths):
        p = _draw_plans(Hq, min(S, pcl), [0, 4, 0, b], (2, 3, 4, 6, 8, 12, 16, 24, 40), 16)
        seqs.append(make_sequence(S, Hq, Hkv, d, min(S, pcl), p, r["amp"], [0, 4, 0, b], device))
        plans.append(p)
        cu.append(cu[-1] + S)
    return _pack("C4 varlen", seqs, cu, pcl, r["tau"], r["mu"], torch.bfloat16, plans)


def decode_case(num_seqs: int = 64, capacity: int = 32768, pcl: int = 2048, device="cpu", seed: int = 6):
    """Generation-time workload: (window Workload, K cache, V cache, q).

    Every sequence owns `capacity` rows of a Llama-3-8B-shaped KV cache (8 KV heads, d 128, bf16).  Its first
    `pcl` rows are a planted window drawn like the layers of config 2 (the masks are built from them); the rest of
    the cache is N(0, 1) noise, which is all a throughput measurement of the gather needs.  q is [num_seqs, 32, 128]."""
    Hq, Hkv, d = 32, 8, 128
    r = CONFIG_RULE[2]
    seqs, plans, cu = [], [], [0]
    for b in range(num_seqs):
        p = _draw_plans(Hq, pcl, [seed, 6, 0, b], (2, 3, 4, 6, 8, 12, 16, 24, 40), 16)
        seqs.append(make_sequence(pcl, Hq, Hkv, d, pcl, p, r["amp"], [seed, 6, 0, b], device))
        plans.append(p)
        cu.append(cu[-1] + pcl)
    win = _pack(f"decode windows {num_seqs} x {pcl}", seqs, cu, pcl, r["tau"], r["mu"], torch.bfloat16, plans)
    gen = _gen([seed, 6, 1], device)
    Kc = torch.randn(num_seqs * capacity, Hkv, d, generator=gen, device=device, dtype=torch.bfloat16)
    Vc = torch.randn(num_seqs * capacity, Hkv, d, generator=gen, device=device, dtype=torch.bfloat16)
    for b in range(num_seqs):
        Kc[b * capacity: b * capacity + pcl] = win.K[b * pcl: (b + 1) * pcl]
        Vc[b * capacity: b * capacity + pcl] = win.V[b * pcl: (b + 1) * pcl]
    q = torch.randn(num_seqs, Hq, d, generator=gen, device=device, dtype=torch.bfloat16)
    return win, Kc, Vc, q


def small_case(S: int, Hq: int, Hkv: int, d: int, pcl: int, seed: int = 1, dtype=torch.bfloat16, device="cpu",
               lengths: Optional[Sequence[int]] = None, tau: float = 0.05, mu: float = 0.8, amp: float = 8.0,
               max_stripes: int = 3) -> Workload:
    """Reduced-size case with the same recipe, for parity tests that visit every row."""
    lengths = list(lengths) if lengths else [S]
    seqs, plans, cu = [], [], [0]
    for b, Sb in enumerate(lengths):
        Lb = min(Sb, pcl)
        p = _draw_plans(Hq, Lb, [seed, 9, 0, b], (2, 3, 4, 8), max_stripes)
        seqs.append(make_sequence(Sb, Hq, Hkv, d, Lb, p, amp, [seed, 9, 0, b], device))
        plans.append(p)
        cu.append(cu[-1] + Sb)
    return _pack(f"small S={lengths}", seqs, cu, pcl, tau, mu, dtype, plans)
