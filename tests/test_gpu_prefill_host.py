"""The host-buffer entry point (uploads, mask construction, attention and downloads pipelined over row chunks)
returns exactly what the two device calls return on the same inputs."""
import pytest
import torch

from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import synth

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
    blob, _ = B.dam_build_masks(Q, K, shape, rule)
    # (the masks keep no key beyond the query either way, so a chunk never needs keys past its end)
    O, lse, scratch = B.dam_sparse_attention(Q, K, V, blob, shape, causal=causal)
    assert B.dam_poll_status(blob) == 0 and B.dam_poll_status(scratch) == 0
    Qh, Kh, Vh = (x.contiguous().pin_memory() for x in (w.Q, w.K, w.V))
    Oh = torch.full(w.Q.shape, 7.0, dtype=dtype).pin_memory()
    lh = torch.full(tuple(lse.shape), 7.0, dtype=torch.float32).pin_memory()
    n = B.dam_prefill_host(Qh, Kh, Vh, shape, rule, Oh, lh, None, DEV)
    ws = torch.empty(n, dtype=torch.uint8, device=DEV)
    for _ in range(2):                                            # the second call reuses the workspace
        B.dam_prefill_host(Qh, Kh, Vh, shape, rule, Oh, lh, ws, DEV, causal=causal)
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
