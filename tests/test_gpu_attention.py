"""Stage-2 parity on the GPU, through the C ABI: with an identical mask, O and LSE must match the
float64 oracle within max-abs 2e-2 / mean-abs 2e-3 (bf16 in, fp32 accumulate) and 1e-3 for LSE."""
import numpy as np
import pytest
import torch

from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = {torch.bfloat16: (2e-2, 2e-3, 1e-3), torch.float32: (1e-4, 1e-5, 1e-5)}


def _shape(w):
    return B.make_shape(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, w.head_dim, w.Q.dtype, DEV)


def _run(w, blob, shape, causal=True, sentinel=False):
    Q, K, V = w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV)
    O = lse = None
    if sentinel:
        # every row of every head must be written: a work item that was dropped would leave the NaN fill behind
        O = torch.full_like(Q, float("nan"))
        lse = torch.full((w.num_q_heads, Q.shape[0]), float("nan"), dtype=torch.float32, device=DEV)
    O, lse, scratch = B.dam_sparse_attention(Q, K, V, blob, shape, causal=causal, O=O, lse=lse)
    assert B.dam_poll_status(scratch) == 0
    # bf16 with head_dim 128 or 64 is served by the tcgen05 kernel, everything else by the CUDA-core kernel
    assert B.attention_ran_on_tensor_cores(scratch) == (w.Q.dtype == torch.bfloat16 and w.head_dim in (64, 128))
    if sentinel:
        _assert_every_row_written(O, lse)
    return O, lse


def _assert_every_row_written(O, lse):
    """No fill value left: O finite everywhere, LSE finite or -inf, and O = 0 exactly on the rows whose LSE is -inf."""
    assert torch.isfinite(O).all(), "rows of O were not written"
    assert not torch.isnan(lse).any() and not torch.isposinf(lse).any(), "rows of LSE were not written"
    empty = torch.isneginf(lse).transpose(0, 1)                       # [T, Hq]
    assert (O[empty] == 0).all()


def _check(w, O, lse, masks, rows_for, heads=None, causal=True, all_ones=False):
    mx, mn, le = TOL[w.Q.dtype]
    worst = [0.0, 0.0, 0.0]
    for b in range(len(w.cu_seqlens) - 1):
        S = w.cu_seqlens[b + 1] - w.cu_seqlens[b]
        if S == 0:
            continue
        for h in (heads if heads is not None else range(w.num_q_heads)):
            e = H.attention_errors(O, lse, w, masks, b, h, rows_for(S), causal=causal, all_ones=all_ones)
            worst = [max(a, c) for a, c in zip(worst, e)]
    assert worst[0] <= mx and worst[1] <= mn and worst[2] <= le, worst
    return worst


def _all_rows(S):
    return list(range(S))


def _sample_rows(L, n_random=256, n_blocks=8):
    """The rows around the window edges and the first row without overlap of columns and diagonals, both edge rows
    of `n_blocks` random 128-row query blocks, and `n_random` random rows."""
    def f(S, L=L):
        rng = np.random.default_rng(S)
        fixed = [0, L - 1, L, L + 1, 2 * L - 2, 2 * L - 1, S - 1, 127, 128, S - 129]
        nq = (S + 127) // 128
        for qb in rng.choice(nq, size=min(nq, n_blocks), replace=False):
            fixed += [int(qb) * 128, min(S - 1, int(qb) * 128 + 127)]
        rows = set(r for r in fixed if 0 <= r < S) | set(int(x) for x in rng.choice(S, size=min(S, n_random), replace=False))
        return sorted(rows)
    return f


HEADS8 = [0, 5, 9, 13, 18, 22, 27, 31]


@pytest.mark.parametrize("lengths,Hq,Hkv,d,dtype,causal", [
    ([512], 2, 2, 64, torch.float32, True),
    ([300, 77, 129], 4, 2, 64, torch.bfloat16, True),
    ([200], 2, 1, 32, torch.float32, False),
    ([640], 4, 1, 128, torch.bfloat16, True),
    ([257, 1, 500], 8, 2, 128, torch.bfloat16, True),
    ([384], 2, 2, 128, torch.bfloat16, False),
])
def test_all_ones_mask_is_dense_attention(lengths, Hq, Hkv, d, dtype, causal):
    w = synth.small_case(0, Hq, Hkv, d, 64, seed=7, dtype=dtype, lengths=lengths, amp=3.0)
    shape = _shape(w)
    blob = B.dam_mask_all_ones(shape, causal, DEV)
    O, lse = _run(w, blob, shape, causal=causal)
    _check(w, O, lse, None, _all_rows, causal=causal, all_ones=True)


def _masked_case(w, rows_for, heads=None, gather=False, sentinel=False):
    shape = _shape(w)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps, gather_columns=gather)
    n = sum(w.num_q_heads * min(S, w.pcl_max) ** 2 for S in shape.lengths)
    dump = torch.zeros(n, dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule, scores_dump=dump)
    assert B.dam_poll_status(blob) == 0
    masks = H.oracle_masks_from_dump(w, dump.cpu().numpy(), heads=heads)      # identical mask on both sides
    O, lse = _run(w, blob, shape, sentinel=sentinel)
    worst = _check(w, O, lse, masks, rows_for, heads=heads)
    return blob, shape, masks, O, lse, worst


def test_config0_every_row():
    w = synth.config0()
    blob, shape, masks, O, lse, worst = _masked_case(w, _all_rows)
    # rows below the window with no matched pattern are empty: O = 0, LSE = -inf (checked inside)
    assert torch.isfinite(O).all()


@pytest.mark.parametrize("lengths,pcl,Hq,Hkv,d,dtype", [
    ([700], 256, 4, 2, 128, torch.bfloat16),
    ([333, 1000, 64], 200, 4, 1, 64, torch.bfloat16),
    ([1500, 130], 256, 8, 2, 128, torch.bfloat16),
    ([513], 300, 2, 2, 32, torch.float32),
    ([2100, 700], 384, 8, 2, 64, torch.bfloat16),            # head_dim 64 on the tensor cores, several tiles and a ragged tail
])
@pytest.mark.parametrize("gather", [False, True])
def test_masked_small_cases_every_row(lengths, pcl, Hq, Hkv, d, dtype, gather):
    w = synth.small_case(0, Hq, Hkv, d, pcl, seed=11, dtype=dtype, lengths=lengths)
    _masked_case(w, _all_rows, gather=gather)


def test_empty_rows_and_no_patterns():
    """mu > 1: nothing matches, every row below the window is empty."""
    w = synth.small_case(0, 4, 2, 128, 128, seed=5, lengths=[600])
    w.mu = 1.5
    blob, shape, masks, O, lse, _ = _masked_case(w, _all_rows)
    assert torch.isneginf(lse[:, 128:]).all() and (O[128:] == 0).all()


@pytest.mark.parametrize("gather", [False, True])
def test_config1_sampled_rows(gather):
    w = synth.config1()
    _masked_case(w, _sample_rows(1024), heads=HEADS8, gather=gather, sentinel=True)


def test_config1_dense_causal_sampled_rows():
    w = synth.config1()
    shape = _shape(w)
    blob = B.dam_mask_all_ones(shape, True, DEV)
    O, lse = _run(w, blob, shape)
    _check(w, O, lse, None, lambda S: [0, 1, 127, 128, 4095, 8191], heads=[3, 30], all_ones=True)


@pytest.mark.parametrize("gather", [False, True])
def test_config4_varlen_sampled_rows(gather):
    w = synth.config4()
    _masked_case(w, _sample_rows(1024), heads=HEADS8, gather=gather, sentinel=True)


def test_config2_layer_sampled_rows():
    """One layer of the 32-layer stack (32768 tokens, PCL 2048), in the launch configuration the benchmark times."""
    w = synth.config2_layer(5, DEV)
    blob, shape, masks, O, lse, worst = _masked_case(w, _sample_rows(2048), heads=HEADS8, gather=True, sentinel=True)
    st = B.dam_mask_stats(blob, shape)
    assert 0.01 <= st["tiles"] / st["causal_tiles"] <= 0.30


def test_config3_sampled_rows():
    """131072 tokens, PCL 4096: sampled rows of a few heads against the oracle over all 131072 keys."""
    w = synth.config3(DEV)
    _masked_case(w, _sample_rows(4096), heads=HEADS8, gather=True, sentinel=True)


def test_gathered_blob_with_small_scratch_reports_error():
    """A blob with gathered-column tiles needs the larger scratch; a scratch that holds some tiles but not all, and
    the 256-byte scratch that is enough for every other blob, are both refused on the device: O and LSE stay as
    they were and the status word says BUFFER_TOO_SMALL."""
    w = synth.small_case(0, 4, 2, 128, 128, seed=4, lengths=[900])
    shape = _shape(w)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, gather_columns=True)
    blob, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule)
    assert B.dam_mask_sizes(shape, rule)[2] > 256
    for nbytes in (256 + 65536, 256):
        small = torch.zeros(256 + 70000, dtype=torch.uint8, device=DEV)[:nbytes]
        O = torch.full_like(w.Q.to(DEV), 7.0)
        O, lse, scr = B.dam_sparse_attention(w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV), blob, shape, scratch=small, O=O)
        torch.cuda.synchronize()
        assert B.dam_poll_status(scr) == 3
        assert (O == 7.0).all()


def test_bounded_wait_times_out_cleanly():
    """A wait that nothing satisfies gives up after its limit, the status word says so, and the device keeps
    working (the next kernel runs and is correct)."""
    status, waited_ns = B.dam_selftest_bounded_wait(DEV, limit_us=20000)
    assert status == 5                                   # DAM_ERR_DEVICE_TIMEOUT
    assert 15e6 <= waited_ns <= 500e6
    w = synth.small_case(0, 4, 2, 128, 128, seed=9, lengths=[300])
    shape = _shape(w)
    blob = B.dam_mask_all_ones(shape, True, DEV)
    O, lse = _run(w, blob, shape)
    _check(w, O, lse, None, _all_rows, all_ones=True)


def test_strided_qkv_views():
    """Q, K, V as views of one fused [T, Hq + 2 Hkv, d] tensor: the strides of dam_shape_t are honoured by the
    TMA descriptors and by the plain kernels."""
    for dtype, d in ((torch.bfloat16, 128), (torch.float32, 64)):
        Hq, Hkv = 4, 2
        w = synth.small_case(0, Hq, Hkv, d, 128, seed=13, dtype=dtype, lengths=[400, 131])
        T = w.Q.shape[0]
        fused = torch.zeros(T, Hq + 2 * Hkv, d, dtype=dtype, device=DEV)
        fused[:, :Hq] = w.Q.to(DEV); fused[:, Hq:Hq + Hkv] = w.K.to(DEV); fused[:, Hq + Hkv:] = w.V.to(DEV)
        Qv, Kv, Vv = fused[:, :Hq], fused[:, Hq:Hq + Hkv], fused[:, Hq + Hkv:]
        st = ((Hq + 2 * Hkv) * d, d)
        shape = B.make_shape(w.cu_seqlens, Hq, Hkv, d, dtype, DEV, q_strides=st, k_strides=st, v_strides=st)
        rule = B.make_rule(w.pcl_max, w.tau, w.mu, gather_columns=True)
        n = sum(Hq * min(S, w.pcl_max) ** 2 for S in shape.lengths)
        dump = torch.zeros(n, dtype=torch.float32, device=DEV)
        blob, _ = B.dam_build_masks(Qv, Kv, shape, rule, scores_dump=dump)
        masks = H.oracle_masks_from_dump(w, dump.cpu().numpy())
        O = torch.empty(T, Hq, d, dtype=dtype, device=DEV)
        O, lse, scr = B.dam_sparse_attention(Qv, Kv, Vv, blob, shape, O=O)
        assert B.dam_poll_status(scr) == 0 and B.dam_poll_status(blob) == 0
        _check(w, O, lse, masks, _all_rows)


@pytest.mark.parametrize("gather", [False, True])
def test_degenerate_lengths(gather):
    """Empty and one-token sequences inside a packed batch, a sequence shorter than a tile, MHA (group 1)."""
    w = synth.small_case(0, 4, 4, 128, 64, seed=17, lengths=[0, 1, 5, 0, 257, 128])
    _masked_case(w, _all_rows, gather=gather)
    shape = _shape(w)
    blob = B.dam_mask_all_ones(shape, True, DEV)
    O, lse = _run(w, blob, shape)
    _check(w, O, lse, None, _all_rows, all_ones=True)


@pytest.mark.parametrize("lengths,Hq,Hkv,d,dtype,gather", [
    ([1024, 300, 700], 8, 2, 128, torch.bfloat16, False),
    ([1536], 4, 1, 128, torch.bfloat16, True),
    ([900, 512], 2, 2, 64, torch.float32, False),
])
def test_chunked_prefill_equals_one_call(lengths, Hq, Hkv, d, dtype, gather):
    """Row ranges: chunks of 256 / 512 rows, with the cache beyond each chunk's end poisoned, give the oracle's
    O and LSE on every row (Sec. 4.3, Case 2, applied to rows that arrive in chunks) and, bit for bit, the output of
    the single call (the arithmetic per row is the same and no row reads a key beyond itself)."""
    w = synth.small_case(0, Hq, Hkv, d, 128, seed=21, dtype=dtype, lengths=lengths)
    shape = _shape(w)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps, gather_columns=gather)
    Q, K, V = w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV)
    dump = torch.zeros(sum(Hq * min(S, w.pcl_max) ** 2 for S in lengths), dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(Q, K, shape, rule, scores_dump=dump)
    masks = H.oracle_masks_from_dump(w, dump.cpu().numpy())
    O_ref, lse_ref, _ = B.dam_sparse_attention(Q, K, V, blob, shape, causal=True)
    O = torch.full_like(O_ref, 7.0)
    lse = torch.full_like(lse_ref, 7.0)
    chunk = 512 if d == 128 else 256
    done = [0] * len(lengths)
    while any(dn < S for dn, S in zip(done, lengths)):
        ranges, Kc, Vc = [], K.clone(), V.clone()
        for b, S in enumerate(lengths):
            r0, r1 = (done[b], min(S, done[b] + chunk)) if done[b] < S else (0, 0)
            ranges.append((r0, r1))
            t0 = w.cu_seqlens[b]
            Kc[t0 + r1: t0 + S] = float("nan")               # keys that have not arrived yet
            Vc[t0 + r1: t0 + S] = float("nan")
            done[b] = max(done[b], r1)
        scratch = B.dam_sparse_attention_rows(Q, Kc, Vc, blob, shape, ranges, O, lse)
        assert B.dam_poll_status(scratch) == 0
    _check(w, O, lse, masks, _all_rows)                      # the chunked output itself against the oracle
    assert torch.equal(O, O_ref)
    assert torch.equal(lse, lse_ref)


def test_row_ranges_leave_other_rows_alone_and_reject_odd_bounds():
    w = synth.small_case(0, 4, 2, 128, 128, seed=22, dtype=torch.bfloat16, lengths=[768, 512])
    shape = _shape(w)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps)
    Q, K, V = w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV)
    blob, _ = B.dam_build_masks(Q, K, shape, rule)
    O_ref, lse_ref, _ = B.dam_sparse_attention(Q, K, V, blob, shape, causal=True)
    O = torch.full_like(O_ref, 7.0)
    lse = torch.full_like(lse_ref, 7.0)
    B.dam_sparse_attention_rows(Q, K, V, blob, shape, [(256, 512), (0, 0)], O, lse)
    assert torch.equal(O[256:512], O_ref[256:512]) and torch.equal(lse[:, 256:512], lse_ref[:, 256:512])
    keep = torch.ones(O.shape[0], dtype=torch.bool, device=DEV)
    keep[256:512] = False
    assert (O[keep] == 7.0).all() and (lse[:, keep] == 7.0).all()
    for bad in ([(128, 512), (0, 0)], [(0, 300), (0, 0)], [(0, 1024), (0, 0)], [(512, 256), (0, 0)]):
        with pytest.raises(B.DamError):
            B.dam_sparse_attention_rows(Q, K, V, blob, shape, bad, O, lse)


@pytest.mark.parametrize("gather", [False, True])
def test_inactive_keys_with_huge_logits(gather):
    """Keys outside every pattern whose logits dwarf the active ones (K rows below the window scaled up): the
    row maximum over all entries of a tile then lies far above the masked one, which is the case the softmax
    must detect (the reference may only follow the masked maximum) and must survive without overflow."""
    w = synth.small_case(0, 4, 2, 128, 128, seed=31, dtype=torch.bfloat16, lengths=[1280, 520])
    rng = np.random.default_rng(5)
    K = w.K.clone()
    for b, S in enumerate([1280, 520]):
        t0 = w.cu_seqlens[b]
        rows = rng.choice(np.arange(128, S), size=(S - 128) // 3, replace=False)
        K[t0 + torch.as_tensor(rows)] *= 12.0                # logits up to a few hundred in either direction
    w.K = K
    if hasattr(w, "_host_qkv"):
        del w._host_qkv
    _, _, _, _, _, worst = _masked_case(w, _sample_rows(128), gather=gather)
    assert all(np.isfinite(worst))
