"""Pins for the attention half of the CPU oracle: masked softmax attention over all keys of a sequence.

Checked against an independent numpy brute force, torch's float64 scaled-dot-product attention (library
routine) and invariants that follow from the definition (Sec. 3 and the last paragraph of Sec. 4.3)."""
import math

import numpy as np
import pytest
import torch

from oracle import dam_oracle as orc


def _rand(S, Hq, Hkv, d, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((S, Hq, d)).astype(np.float32),
            rng.standard_normal((S, Hkv, d)).astype(np.float32),
            rng.standard_normal((S, Hkv, d)).astype(np.float32))


def _numpy_attention(q, k, v, mask, scale):
    s = (q.astype(np.float64) @ k.astype(np.float64).T) * scale
    s = np.where(mask.astype(bool), s, -np.inf)
    m = s.max(1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(1, keepdims=True)
    return (e / l) @ v.astype(np.float64), (m + np.log(l))[:, 0]


def test_all_ones_mask_is_dense_causal_attention():
    S, Hq, Hkv, d = 50, 4, 2, 16
    Q, K, V = _rand(S, Hq, Hkv, d, 0)
    rows = list(range(S))
    causal = np.tril(np.ones((S, S), np.uint8))
    for h in range(Hq):
        O, lse = orc.attention(Q, K, V, [0, S], 0, h, rows, None, causal=True)
        O2, lse2 = _numpy_attention(Q[:, h], K[:, h // 2], V[:, h // 2], causal, 1 / math.sqrt(d))
        assert np.allclose(O, O2, atol=1e-13) and np.allclose(lse, lse2, atol=1e-13)
        # same thing with an explicit all-ones mask
        O3, lse3 = orc.attention(Q, K, V, [0, S], 0, h, rows, None, causal=True,
                                 mask_rows=np.ones((S, S), np.uint8))
        assert np.array_equal(O, O3) and np.array_equal(lse, lse3)
        # torch float64 library routine (GQA: KV head h // 2)
        tq = torch.from_numpy(Q[:, h]).double()[None, None]
        tk = torch.from_numpy(K[:, h // 2]).double()[None, None]
        tv = torch.from_numpy(V[:, h // 2]).double()[None, None]
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0, 0].numpy()
        assert np.allclose(O, ref, atol=1e-12)


def test_non_causal_full_attention():
    S, d = 33, 8
    Q, K, V = _rand(S, 1, 1, d, 1)
    O, lse = orc.attention(Q, K, V, [0, S], 0, 0, list(range(S)), None, causal=False)
    O2, lse2 = _numpy_attention(Q[:, 0], K[:, 0], V[:, 0], np.ones((S, S)), 1 / math.sqrt(d))
    assert np.allclose(O, O2, atol=1e-13) and np.allclose(lse, lse2, atol=1e-13)


def test_masked_attention_matches_library_with_attn_mask():
    S, d = 64, 16
    Q, K, V = _rand(S, 1, 1, d, 2)
    rng = np.random.default_rng(3)
    mask = np.tril(rng.random((S, S)) < 0.3).astype(np.uint8)
    mask[np.arange(S), np.arange(S)] = 1            # no empty rows for the library comparison
    O, lse = orc.attention(Q, K, V, [0, S], 0, 0, list(range(S)), None, causal=True, mask_rows=mask)
    tq, tk, tv = (torch.from_numpy(x[:, 0]).double()[None, None] for x in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask).bool())
    assert np.allclose(O, ref[0, 0].numpy(), atol=1e-12)
    O2, lse2 = _numpy_attention(Q[:, 0], K[:, 0], V[:, 0], mask, 1 / math.sqrt(d))
    assert np.allclose(lse, lse2, atol=1e-13)


def test_invariants_one_key_uniform_and_masked_values():
    S, d = 40, 8
    Q, K, V = _rand(S, 1, 1, d, 4)
    scale = 1 / math.sqrt(d)
    # one active key: O = v_j and LSE = the logit itself
    mask = np.zeros((S, S), np.uint8)
    mask[np.arange(S), np.arange(S) // 2] = 1
    O, lse = orc.attention(Q, K, V, [0, S], 0, 0, list(range(S)), None, causal=True, mask_rows=mask)
    for i in range(S):
        j = i // 2
        assert np.allclose(O[i], V[j, 0].astype(np.float64), atol=1e-15)
        assert abs(lse[i] - scale * float(Q[i, 0].astype(np.float64) @ K[j, 0].astype(np.float64))) < 1e-13
    # Q = 0: uniform weights over the active keys, LSE = ln(count)
    Q0 = np.zeros_like(Q)
    rng = np.random.default_rng(5)
    mask = np.tril(rng.random((S, S)) < 0.4).astype(np.uint8)
    mask[:, 0] = 1
    O, lse = orc.attention(Q0, K, V, [0, S], 0, 0, list(range(S)), None, causal=True, mask_rows=mask)
    for i in range(S):
        act = np.flatnonzero(mask[i])
        assert np.allclose(O[i], V[act, 0].astype(np.float64).mean(0), atol=1e-14)
        assert abs(lse[i] - math.log(len(act))) < 1e-14
    # masked keys contribute exactly zero: changing their values changes nothing
    O1, l1 = orc.attention(Q, K, V, [0, S], 0, 0, list(range(S)), None, causal=True, mask_rows=mask)
    V2, K2 = V.copy(), K.copy()
    dead = np.flatnonzero(mask.sum(0) == 0)
    V2[dead] = 1e6
    K2[dead] = 1e3
    O2, l2 = orc.attention(Q, K2, V2, [0, S], 0, 0, list(range(S)), None, causal=True, mask_rows=mask)
    assert np.array_equal(O1, O2) and np.array_equal(l1, l2)


def test_empty_rows_give_zero_and_minus_inf():
    S, d = 10, 4
    Q, K, V = _rand(S, 1, 1, d, 6)
    mask = np.zeros((S, S), np.uint8)
    mask[3, 1] = 1
    O, lse = orc.attention(Q, K, V, [0, S], 0, 0, list(range(S)), None, causal=True, mask_rows=mask)
    assert np.all(O[[0, 1, 2, 4, 9]] == 0.0)
    assert np.all(np.isneginf(lse[[0, 1, 2, 4, 9]]))
    assert np.isfinite(lse[3])


def test_rows_subset_and_varlen_offsets():
    """Rows are indices inside the chosen sequence of a packed batch; keys never cross sequences."""
    lens = [7, 20, 13]
    cu = np.concatenate([[0], np.cumsum(lens)]).tolist()
    T, d = cu[-1], 8
    Q, K, V = _rand(T, 2, 1, d, 7)
    for b, S in enumerate(lens):
        rows = [0, S // 2, S - 1]
        O, lse = orc.attention(Q, K, V, cu, b, 1, rows, None, causal=True)
        sl = slice(cu[b], cu[b + 1])
        O2, lse2 = _numpy_attention(Q[sl, 1], K[sl, 0], V[sl, 0], np.tril(np.ones((S, S))), 1 / math.sqrt(d))
        assert np.allclose(O, O2[rows], atol=1e-13) and np.allclose(lse, lse2[rows], atol=1e-13)


def test_build_masks_per_sequence_and_gqa():
    """Masks are built per sequence from that sequence's first L tokens, per query head, with the KV head
    of the group."""
    from paper_2506_11104_b200 import synth
    w = synth.small_case(0, 4, 2, 64, 64, seed=3, dtype=torch.float32, lengths=[100, 48, 200])
    Q, K = w.Q.numpy(), w.K.numpy()
    masks = orc.build_masks(Q, K, w.cu_seqlens, w.pcl_max, w.tau, w.mu)
    assert [m[0].L for m in masks] == [64, 48, 64]
    b, h = 2, 3
    t0 = w.cu_seqlens[b]
    P = orc.window_probs(np.ascontiguousarray(Q[t0:t0 + 64, h]), np.ascontiguousarray(K[t0:t0 + 64, h // 2]),
                         64, 1 / 8.0)
    ref = orc.head_mask_from_probs(P, 200, w.tau, w.mu)
    assert np.array_equal(masks[b][h].M, ref.M) and np.array_equal(masks[b][h].D, ref.D)
