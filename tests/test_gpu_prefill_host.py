"""The host-buffer entry point (uploads, mask construction, attention and downloads pipelined over row chunks):
its O and LSE against the float64 oracle (masks from the shared fp32 score tensor), and bit for bit against the two
device calls on the same inputs."""
import numpy as np
import pytest
import torch

from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import synth
from tests import helpers as H

TOL = {torch.bfloat16: (2e-2, 2e-3, 1e-3), torch.float32: (1e-4, 1e-5, 1e-5)}


def _oracle_check(w, Oh, lh, masks, causal):
    """Sampled rows of every (sequence, head) of the host-side result against the oracle (Sec. 4.3)."""
    mx, mn, le = TOL[w.Q.dtype]
    for b in range(len(w.cu_seqlens) - 1):
        S = w.cu_seqlens[b + 1] - w.cu_seqlens[b]
        rng = np.random.default_rng(S)
        L = min(S, w.pcl_max)
        fixed = [0, L - 1, L, L + 1, 2 * L - 2, 2 * L - 1, S - 1, 255, 256, 2047, 2048, 4095, 4096]
        rows = sorted(set(r for r in fixed if 0 <= r < S) | set(int(x) for x in rng.choice(S, size=min(S, 256), replace=False)))
        for h in range(w.num_q_heads):
            e = H.attention_errors(Oh, lh, w, masks, b, h, rows, causal=causal)
            assert e[0] <= mx and e[1] <= mn and e[2] <= le, (b, h, e)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("lengths,Hq,Hkv,d,dtype,pcl,gather", [
    ([9000], 4, 2, 128, torch.bfloat16, 512, True),              # one sequence, three chunks, ragged end
    ([5000, 300, 4500, 130], 4, 1, 128, torch.bfloat16, 384, True),   # chunks that span sequences
    ([4200, 4100], 2, 2, 128, torch.bfloat16, 256, False),
    ([700, 260], 2, 1, 64, torch.float32, 128, False),           # CUDA-core path, one chunk
])
@pytest.mark.parametrize("causal", [True, False])
def test_prefill_host_equals_device_calls(lengths, Hq, Hkv, d, dtype, pcl, gather, causal):
    w = synth.small_case(0, Hq, Hkv, d, pcl, seed=21, dtype=dtype, lengths=lengths)
    shape = B.make_shape(w.cu_seqlens, Hq, Hkv, d, dtype, DEV)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps, gather_columns=gather)
    Q, K, V = w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV)
    dump = torch.zeros(sum(Hq * min(S, pcl) ** 2 for S in lengths), dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(Q, K, shape, rule, scores_dump=dump)
    masks = H.oracle_masks_from_dump(w, dump.cpu().numpy())
    # (the masks keep no key beyond the query either way, so a chunk never needs keys past its end)
    O, lse, scratch = B.dam_sparse_attention(Q, K, V, blob, shape, causal=causal)
    assert B.dam_poll_status(blob) == 0 and B.dam_poll_status(scratch) == 0
    Qh, Kh, Vh = (x.contiguous().pin_memory() for x in (w.Q, w.K, w.V))
    Oh = torch.full(w.Q.shape, 7.0, dtype=dtype).pin_memory()
    lh = torch.full(tuple(lse.shape), 7.0, dtype=torch.float32).pin_memory()
    n = B.dam_prefill_host(Qh, Kh, Vh, shape, rule, Oh, lh, None, DEV)
    ws = torch.empty(n, dtype=torch.uint8, device=DEV)
    for it in range(2):                                           # the second call reuses the workspace
        B.dam_prefill_host(Qh, Kh, Vh, shape, rule, Oh, lh, ws, DEV, causal=causal)
        if it == 0:
            _oracle_check(w, Oh, lh, masks, causal)
        assert torch.equal(Oh.view(torch.uint8), O.cpu().view(torch.uint8))
        assert torch.equal(lh.view(torch.uint8), lse.cpu().view(torch.uint8))
        Oh.fill_(7.0); lh.fill_(7.0)


def test_prefill_host_workspace_too_small():
    w = synth.small_case(0, 2, 1, 64, 64, seed=2, dtype=torch.bfloat16, lengths=[300])
    shape = B.make_shape(w.cu_seqlens, 2, 1, 64, torch.bfloat16, DEV)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps)
    Oh = torch.empty(w.Q.shape, dtype=torch.bfloat16)
    lh = torch.empty(2, 300, dtype=torch.float32)
    n = B.dam_prefill_host(w.Q, w.K, w.V, shape, rule, Oh, lh, None, DEV)
    ws = torch.empty(n - 256, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.DamError):
        B.dam_prefill_host(w.Q, w.K, w.V, shape, rule, Oh, lh, ws, DEV)


def test_prefill_host_with_a_poisoned_workspace():
    """A chunk that ends at a sequence end inside a 128-key tile makes that tile's K / V rows reach into tokens
    of the next sequence that arrive with a later chunk (here the windows are shorter than a tile, so they are not
    among the rows that go up first).  Their probabilities are zero, and the workspace starts out as NaN bit
    patterns: the result must still be the device calls' result, bit for bit, and pass the oracle."""
    lengths, Hq, Hkv, d, pcl = [2100, 2300, 2500], 4, 2, 128, 48
    w = synth.small_case(0, Hq, Hkv, d, pcl, seed=23, dtype=torch.bfloat16, lengths=lengths)
    shape = B.make_shape(w.cu_seqlens, Hq, Hkv, d, torch.bfloat16, DEV)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps, gather_columns=True)
    Q, K, V = w.Q.to(DEV), w.K.to(DEV), w.V.to(DEV)
    dump = torch.zeros(sum(Hq * min(S, pcl) ** 2 for S in lengths), dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(Q, K, shape, rule, scores_dump=dump)
    masks = H.oracle_masks_from_dump(w, dump.cpu().numpy())
    O, lse, scratch = B.dam_sparse_attention(Q, K, V, blob, shape, causal=True)
    Qh, Kh, Vh = (x.contiguous().pin_memory() for x in (w.Q, w.K, w.V))
    Oh = torch.full(w.Q.shape, 7.0, dtype=torch.bfloat16).pin_memory()
    lh = torch.full(tuple(lse.shape), 7.0, dtype=torch.float32).pin_memory()
    n = B.dam_prefill_host(Qh, Kh, Vh, shape, rule, Oh, lh, None, DEV)
    ws = torch.full((n,), 0xFF, dtype=torch.uint8, device=DEV)       # every bf16 of the workspace is a NaN
    B.dam_prefill_host(Qh, Kh, Vh, shape, rule, Oh, lh, ws, DEV)
    assert torch.isfinite(Oh.float()).all()
    assert torch.equal(Oh.view(torch.uint8), O.cpu().view(torch.uint8))
    assert torch.equal(lh.view(torch.uint8), lse.cpu().view(torch.uint8))
    _oracle_check(w, Oh, lh, masks, True)
