"""Host-only checks of the C ABI: the library loads without a GPU, exports every function that
include/dam.h declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest
import torch

from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import build as dam_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    dam_build.build()


def test_exports_match_header():
    text = open(os.path.join(ROOT, "include", "dam.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(dam_[a-z_0-9]+)\s*\(", text))
    assert declared == set(B.EXPORTS)
    lib = B.lib()
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings():
    assert B.dam_version() >= 1000
    assert B.dam_status_string(0) == "ok"
    assert "timed out" in B.dam_status_string(5)
    assert B.dam_status_string(99) == "unknown status"


def test_mask_sizes_bounds():
    sh = B.make_shape([0, 131072], 32, 8, 128, torch.bfloat16)
    rule = B.make_rule(4096, 0.05, 0.8)
    mb, sb, ab = B.dam_mask_sizes(sh, rule)
    true_bits = 32 * 4096 * 4096 // 8
    assert true_bits < mb < true_bits + 64 * 2 ** 20       # tile lists and tables stay small
    assert sb > 0 and ab >= 256
    mb1, sb1, _ = B.dam_mask_sizes(sh, None, True)
    assert sb1 == 0 and mb1 > 4 * 32 * (1024 * 1025 // 2)
    # varlen: sizes add up per sequence
    sh2 = B.make_shape([0, 4096, 20480, 53248, 118784], 32, 8, 128, torch.bfloat16)
    assert B.dam_mask_sizes(sh2, B.make_rule(1024, 0.05, 0.8))[0] > 4 * 32 * 1024 * 1024 // 8


@pytest.mark.parametrize("mutate,code", [
    (lambda s, r: setattr(s.c, "struct_size", 8), 1),
    (lambda s, r: setattr(s.c, "num_kv_heads", 3), 1),
    (lambda s, r: setattr(s.c, "head_dim", 12), 1),
    (lambda s, r: setattr(s.c, "head_dim", 512), 2),
    (lambda s, r: setattr(s.c, "total_tokens", 5), 1),
    (lambda s, r: setattr(s.c, "max_seqlen", 5), 1),
    (lambda s, r: setattr(s.c, "q_stride_tok", 130), 1),
    (lambda s, r: setattr(r, "tau", 0.0), 1),
    (lambda s, r: setattr(r, "eps", 0.0), 1),
    (lambda s, r: setattr(r, "pcl_max", 0), 1),
    (lambda s, r: setattr(r, "lambda_", float("nan")), 1),
    (lambda s, r: setattr(r, "transform", 9), 1),
    (lambda s, r: setattr(r, "transform", -1), 1),
    (lambda s, r: setattr(r, "min_support", 0), 1),
    (lambda s, r: setattr(r, "struct_size", 4), 1),
])
def test_invalid_arguments_rejected_on_host(mutate, code):
    sh = B.make_shape([0, 300, 700], 4, 2, 128, torch.bfloat16)
    rule = B.make_rule(256, 0.3, 0.8)
    mutate(sh, rule)
    with pytest.raises(B.DamError) as e:
        B.dam_mask_sizes(sh, rule)
    assert e.value.code == code


def test_null_and_misaligned_pointers_rejected_before_any_launch():
    sh = B.make_shape([0, 256], 2, 2, 64, torch.float32)
    rule = B.make_rule(128, 0.3, 0.8)
    lib = B.lib()
    null = ctypes.c_void_p(0)
    rc = lib.dam_build_masks(null, null, sh.ref, ctypes.byref(rule), null, ctypes.c_size_t(0), null,
                             ctypes.c_size_t(0), null, null)
    assert rc == 1
    fake = ctypes.c_void_p(0x1000)          # aligned, never dereferenced: the size check fires first
    rc = lib.dam_build_masks(fake, fake, sh.ref, ctypes.byref(rule), fake, ctypes.c_size_t(16), fake,
                             ctypes.c_size_t(16), null, null)
    assert rc == 3
    odd = ctypes.c_void_p(0x1001)
    rc = lib.dam_sparse_attention(odd, fake, fake, fake, sh.ref, 1, 1, ctypes.c_float(0.0), fake, fake, fake,
                                  ctypes.c_size_t(256), null)
    assert rc == 1
    rc = lib.dam_sparse_attention(fake, fake, fake, fake, sh.ref, 1, 2, ctypes.c_float(0.0), fake, fake, fake,
                                  ctypes.c_size_t(256), null)
    assert rc == 1                            # gqa_group does not match the shape
    n = ctypes.c_size_t(0)
    rc = lib.dam_prefill_host(null, null, null, sh.ref, ctypes.byref(rule), 1, null, null, null, ctypes.byref(n), null)
    assert rc == 0 and n.value > 0            # size query only


def test_per_device_table_keeps_one_record_per_ordinal():
    """The table behind the tensor-core launches (device properties and one-off set-up steps per device ordinal),
    driven with a fake device query for two fake ordinals and from several threads at once."""
    rc, sm, (queries, setups) = B.dam_selftest_device_table([0, 1, 0, 1, 1, 0])
    assert rc == 0 and sm == [100, 101, 100, 101, 101, 100]
    assert queries == 2 and setups == 2                      # once per device, not once per process or per call
    rc, sm, (queries, setups) = B.dam_selftest_device_table([5, 64, -1, 5])
    assert rc == 1 and sm == [105, -1, -1, 105] and queries == 1 and setups == 1
    import threading
    results = []
    ts = [threading.Thread(target=lambda k=k: results.append(B.dam_selftest_device_table([k % 3, (k + 1) % 3] * 50)))
          for k in range(8)]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    assert len(results) == 8 and all(r[0] == 0 and r[2] == (2, 2) for r in results)
