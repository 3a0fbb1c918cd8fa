"""dam_build_masks_static: the variant of stage 1 for callers that cannot allocate device memory (a server
whose memory pool owns the whole GPU, a loop that must not call cudaMalloc).  It takes its scratch from a
fixed array inside the library.  Checked here through the C ABI against dam_build_masks, bit for bit, on
two calls in a row with different inputs (the second call meets the first call's leftovers in the array)."""
import pytest
import torch

from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _blob_sections(blob):
    mb = B.MaskBlob(blob)
    out = [mb.seqs.tobytes(), mb.tile_ptr.tobytes(), mb.tiles.tobytes(), int(mb.hdr["total_tiles"]),
           int(mb.hdr["full_tiles"]), int(mb.hdr["bytes_used"])]
    for b in range(int(mb.hdr["num_seqs"])):
        for h in range(int(mb.hdr["num_q_heads"])):
            out.extend(x.tobytes() for x in mb.pattern_bits(b, h))
            out.append(mb.true_mask(b, h).tobytes())
    # the work list is an unordered-within-equal-keys permutation: compare it as a set
    out.append(sorted(tuple(int(v) for v in it) for it in mb.items))
    return out


def test_static_scratch_matches_regular_entry_point_twice_in_a_row():
    assert B.dam_static_scratch_bytes() == 8 << 20
    cases = [synth.small_case(0, 8, 2, 128, 256, seed=21, lengths=[900, 300]),
             synth.small_case(0, 4, 4, 64, 200, seed=22, lengths=[513], dtype=torch.float32)]
    for w in cases:                      # two calls in a row, different shapes and dtypes
        shape = B.make_shape(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, w.head_dim, w.Q.dtype, DEV)
        rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps)
        Q, K = w.Q.to(DEV), w.K.to(DEV)
        ref, _ = B.dam_build_masks(Q, K, shape, rule)
        mb, _, _ = B.dam_mask_sizes(shape, rule)
        mask = torch.empty(mb, dtype=torch.uint8, device=DEV)       # the caller still owns inputs and outputs
        # the first call on a device looks up the array's address (and the driver may load kernels it has not
        # run yet): that is the documented set-up call.  From then on the free memory the driver reports must
        # not move across a call: torch's own counters would not see a cudaMalloc made inside the library.
        B.dam_build_masks_static(Q, K, shape, rule, mask)
        mask.zero_()                                                 # (torch loads its own fill kernel on first use)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info(DEV)
        B.dam_build_masks_static(Q, K, shape, rule, mask)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(DEV)
        assert free_after == free_before
        assert B.dam_poll_status(mask) == 0 and B.dam_poll_status(ref) == 0
        assert _blob_sections(mask) == _blob_sections(ref)
    # same inputs again: the array now holds this shape's leftovers
    B.dam_build_masks_static(Q, K, shape, rule, mask)
    torch.cuda.synchronize()
    assert _blob_sections(mask) == _blob_sections(ref)


def test_static_scratch_rejects_oversized_shapes():
    # 8 sequences of 131072 tokens x 32 heads at PCL 4096 need far more than 8 MiB of scratch
    cu = [131072 * i for i in range(9)]
    shape = B.make_shape(cu, 32, 8, 128, torch.bfloat16, DEV)
    rule = B.make_rule(4096, 0.05, 0.8)
    need = B.dam_mask_sizes(shape, rule)[1]
    assert need > B.dam_static_scratch_bytes()
    dummy = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(B.DamError) as e:
        B.dam_build_masks_static(dummy, dummy, shape, rule, dummy)
    assert e.value.code == 3
