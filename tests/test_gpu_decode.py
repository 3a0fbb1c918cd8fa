"""Generation-time attention (one new token per sequence against a KV cache, keys chosen by the stored
patterns) against the float64 oracle: the oracle computes row i of the extended mask from (M, D, V) and dense
masked attention of that row over keys 0..i."""
import numpy as np
import pytest
import torch

from oracle import dam_oracle as orc
from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {torch.bfloat16: (2e-2, 2e-3, 1e-3), torch.float32: (1e-4, 1e-5, 1e-5)}


def _build(w, build_lengths):
    """Blob + oracle masks built from the first build_lengths[b] tokens of every sequence of the cache."""
    Hq, Hkv, d = w.num_q_heads, w.num_kv_heads, w.head_dim
    idx = torch.cat([torch.arange(w.cu_seqlens[b], w.cu_seqlens[b] + n) for b, n in enumerate(build_lengths)])
    Qb, Kb = w.Q[idx].contiguous().to(DEV), w.K[idx].contiguous().to(DEV)
    cu = [0] + list(np.cumsum(build_lengths))
    shape = B.make_shape(cu, Hq, Hkv, d, w.Q.dtype, DEV)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps)
    n = sum(Hq * min(S, w.pcl_max) ** 2 for S in build_lengths)
    dump = torch.zeros(n, dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(Qb, Kb, shape, rule, scores_dump=dump)
    assert B.dam_poll_status(blob) == 0
    P = H.split_dump(dump.cpu().numpy(), build_lengths, Hq, w.pcl_max)
    masks = [[orc.head_mask_from_probs(np.ascontiguousarray(P[b][h]), S, w.tau, w.mu, w.lam, w.eps)
              for h in range(Hq)] for b, S in enumerate(build_lengths)]
    return blob, masks


def _decode_and_check(w, blob, masks, positions):
    Hq, Hkv, d = w.num_q_heads, w.num_kv_heads, w.head_dim
    nb = len(w.cu_seqlens) - 1
    cache = B.make_shape(w.cu_seqlens, Hq, Hkv, d, w.Q.dtype, DEV)
    K, V = w.K.to(DEV), w.V.to(DEV)
    q = torch.stack([w.Q[w.cu_seqlens[b] + positions[b]] for b in range(nb)]).contiguous().to(DEV)
    pos = torch.tensor(positions, dtype=torch.int32, device=DEV)
    O, lse, scratch = B.dam_decode_attention(q, K, V, blob, cache, pos)
    assert B.dam_poll_status(scratch) == 0
    Qh, Kh, Vh = H.host_qkv(w)
    mx, mn, le = TOL[w.Q.dtype]
    g = Hq // Hkv
    scale = 1.0 / np.sqrt(d)
    errs = []
    for b in range(nb):
        i = positions[b]
        t0 = w.cu_seqlens[b]
        for h in range(Hq):
            hm = masks[b][h]
            row = orc.extended_rows(hm.M, hm.D, hm.V, max(i + 1, hm.L), [i])[:, :i + 1]   # row i over keys 0..i
            O_ref, lse_ref = orc.attention_rows(Qh[t0:t0 + i + 1, h, :], Kh[t0:t0 + i + 1, h // g, :],
                                                Vh[t0:t0 + i + 1, h // g, :], [i], row, True, scale)
            o = O[b, h].double().cpu().numpy()
            l = float(lse[b, h])
            if np.isfinite(lse_ref[0]):
                errs.append((np.abs(o - O_ref[0]).max(), np.abs(o - O_ref[0]).mean(), abs(l - lse_ref[0])))
            else:
                assert l == -np.inf and not o.any()
    worst = np.max(np.array(errs), axis=0) if errs else np.zeros(3)
    assert worst[0] <= mx and worst[1] <= mn and worst[2] <= le, worst


@pytest.mark.parametrize("cache_lengths,build_lengths,Hq,Hkv,d,dtype,pcl", [
    ([512], [512], 2, 2, 64, torch.float32, 128),
    ([1024, 700], [512, 700], 8, 2, 128, torch.bfloat16, 128),
    ([900], [300], 4, 1, 64, torch.bfloat16, 96),
    ([640, 640, 130], [640, 200, 130], 4, 2, 128, torch.float32, 160),
    ([700], [700], 2, 2, 128, torch.bfloat16, 128),          # one head per KV head on the grouped tensor-core kernel
    ([5000], [5000], 8, 1, 64, torch.bfloat16, 2112),        # eight heads per KV head; 132 pattern words: two rounds
    ([600], [600], 16, 1, 64, torch.bfloat16, 96),           # sixteen heads per KV head: the one-head-per-block kernel
])
def test_decode_matches_oracle(cache_lengths, build_lengths, Hq, Hkv, d, dtype, pcl):
    w = synth.small_case(0, Hq, Hkv, d, pcl, seed=11, dtype=dtype, lengths=cache_lengths)
    blob, masks = _build(w, build_lengths)
    per_seq = []
    for cap, Sb in zip(cache_lengths, build_lengths):
        L = min(Sb, pcl)
        cand = [0, 5, L - 1, L, L + 1, 2 * L - 2, 2 * L - 1, 2 * L, Sb - 1, Sb, (Sb + cap) // 2, cap - 1]
        per_seq.append(sorted(set(min(max(c, 0), cap - 1) for c in cand)))
    for k in range(max(len(p) for p in per_seq)):
        _decode_and_check(w, blob, masks, [p[min(k, len(p) - 1)] for p in per_seq])


def test_decode_agrees_with_prefill_rows():
    """The same rows through the tile-list kernel and through the pattern-walking kernel."""
    w = synth.small_case(0, 8, 2, 128, 128, seed=5, dtype=torch.bfloat16, lengths=[768, 400])
    shape = B.make_shape(w.cu_seqlens, 8, 2, 128, torch.bfloat16, DEV)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps)
    Q, K, V = w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV)
    blob, _ = B.dam_build_masks(Q, K, shape, rule)
    O, lse, _ = B.dam_sparse_attention(Q, K, V, blob, shape, causal=True)
    for positions in ([767, 399], [128, 127], [255, 256], [300, 1]):
        q = torch.stack([Q[w.cu_seqlens[b] + p] for b, p in enumerate(positions)]).contiguous()
        pos = torch.tensor(positions, dtype=torch.int32, device=DEV)
        Od, lsed, scratch = B.dam_decode_attention(q, K, V, blob, shape, pos)
        assert B.dam_poll_status(scratch) == 0
        for b, p in enumerate(positions):
            t = w.cu_seqlens[b] + p
            assert (Od[b].float() - O[t].float()).abs().max().item() <= 2e-2
            a, c = lsed[b], lse[:, t]
            fin = torch.isfinite(c)
            assert torch.equal(torch.isfinite(a), fin)
            assert (a[fin] - c[fin]).abs().max().item() <= 1e-3 if fin.any() else True


def test_decode_rejects_position_outside_cache():
    w = synth.small_case(0, 2, 1, 64, 64, seed=3, dtype=torch.bfloat16, lengths=[256, 256])
    blob, _ = _build(w, [256, 256])
    cache = B.make_shape(w.cu_seqlens, 2, 1, 64, torch.bfloat16, DEV)
    q = torch.ones(2, 2, 64, dtype=torch.bfloat16, device=DEV)
    pos = torch.tensor([100, 256], dtype=torch.int32, device=DEV)            # second one is past the capacity
    O, lse, scratch = B.dam_decode_attention(q, w.K.to(DEV), w.V.to(DEV), blob, cache, pos)
    assert B.dam_poll_status(scratch) == 1                                   # DAM_ERR_INVALID_ARGUMENT
    assert not O[1].float().abs().any() and torch.isneginf(lse[1]).all()
    assert torch.isfinite(lse[0]).any()
