"""Thin ctypes binding of the C ABI in ``include/dam.h``.

Argument marshalling only: every step of the path runs inside the CUDA library.  PyTorch is used for
device memory and streams.  There is no CPU fallback: if ``libdam_b200.so`` is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdam_b200.so")

DAM_BF16, DAM_F32 = 0, 1
STATUS = {0: "DAM_OK", 1: "DAM_ERR_INVALID_ARGUMENT", 2: "DAM_ERR_UNSUPPORTED", 3: "DAM_ERR_BUFFER_TOO_SMALL",
          4: "DAM_ERR_CUDA", 5: "DAM_ERR_DEVICE_TIMEOUT", 6: "DAM_ERR_INTERNAL"}

EXPORTS = ["dam_version", "dam_status_string", "dam_mask_sizes", "dam_build_masks", "dam_build_masks_from_scores",
           "dam_mask_all_ones", "dam_sparse_attention", "dam_mask_stats", "dam_mask_expand_rows", "dam_poll_status",
           "dam_prefill_host", "dam_build_masks_static", "dam_static_scratch_bytes", "dam_selftest_bounded_wait",
           "dam_decode_attention", "dam_sparse_attention_rows", "dam_capture_accumulate", "dam_capture_average",
           "dam_selftest_device_table"]


class DamError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)}")


class dam_shape_t(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("num_seqs", ctypes.c_int32),
                ("cu_seqlens_host", ctypes.c_void_p), ("cu_seqlens_dev", ctypes.c_void_p),
                ("total_tokens", ctypes.c_int32), ("max_seqlen", ctypes.c_int32),
                ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("q_stride_tok", ctypes.c_int64), ("q_stride_head", ctypes.c_int64),
                ("k_stride_tok", ctypes.c_int64), ("k_stride_head", ctypes.c_int64),
                ("v_stride_tok", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
                ("o_stride_tok", ctypes.c_int64), ("o_stride_head", ctypes.c_int64)]


class dam_rule_t(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("pcl_max", ctypes.c_int32), ("tau", ctypes.c_float),
                ("mu", ctypes.c_float), ("lambda_", ctypes.c_float), ("eps", ctypes.c_float),
                ("softmax_scale", ctypes.c_float), ("min_support", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("transform", ctypes.c_int32)]


TRANSFORMS = {"boxcox": 0, "log": 1, "sqrt": 2, "arcsinh": 3, "yeo_johnson": 4, "average": 5, "zscore": 6, "minmax": 7, "sum": 8}


_lib = None


def lib():
    """The loaded shared library; raises if it was not built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_11104_b200.build` "
                               "(there is no fallback path)")
        _lib = ctypes.CDLL(LIB_PATH)
        _lib.dam_version.restype = ctypes.c_int32
        _lib.dam_status_string.restype = ctypes.c_char_p
        _lib.dam_status_string.argtypes = [ctypes.c_int]
        for name in EXPORTS[2:]:
            getattr(_lib, name).restype = ctypes.c_int
        _lib.dam_static_scratch_bytes.restype = ctypes.c_size_t
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise DamError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


@dataclass
class Shape:
    """Python-side owner of a dam_shape_t and the cu_seqlens buffers it points to."""
    c: dam_shape_t
    cu_host: np.ndarray
    cu_dev: Optional[torch.Tensor]
    lengths: List[int]

    @property
    def ref(self):
        return ctypes.byref(self.c)


def make_shape(cu_seqlens: Sequence[int], Hq: int, Hkv: int, d: int, dtype: torch.dtype, device=None,
               q_strides=None, k_strides=None, v_strides=None, o_strides=None) -> Shape:
    cu_host = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    cu_dev = torch.from_numpy(cu_host.copy()).to(device) if device is not None else None
    lengths = [int(b - a) for a, b in zip(cu_host[:-1], cu_host[1:])]
    s = dam_shape_t()
    s.struct_size = ctypes.sizeof(dam_shape_t)
    s.num_seqs = len(lengths)
    s.cu_seqlens_host = cu_host.ctypes.data
    s.cu_seqlens_dev = cu_dev.data_ptr() if cu_dev is not None else 1   # non-null placeholder for host-only calls
    s.total_tokens = int(cu_host[-1])
    s.max_seqlen = max(lengths) if lengths else 0
    s.num_q_heads, s.num_kv_heads, s.head_dim = Hq, Hkv, d
    s.dtype = DAM_BF16 if dtype == torch.bfloat16 else DAM_F32
    qs = q_strides or (Hq * d, d)
    ks = k_strides or (Hkv * d, d)
    vs = v_strides or (Hkv * d, d)
    os_ = o_strides or (Hq * d, d)
    s.q_stride_tok, s.q_stride_head = qs
    s.k_stride_tok, s.k_stride_head = ks
    s.v_stride_tok, s.v_stride_head = vs
    s.o_stride_tok, s.o_stride_head = os_
    return Shape(c=s, cu_host=cu_host, cu_dev=cu_dev, lengths=lengths)


DAM_RULE_GATHER_COLUMNS = 1


def make_rule(pcl_max: int, tau: float, mu: float, lam: float = 0.5, eps: float = 1e-8,
              softmax_scale: float = 0.0, min_support: int = 1, gather_columns: bool = False,
              transform: str = "boxcox") -> dam_rule_t:
    r = dam_rule_t()
    r.struct_size = ctypes.sizeof(dam_rule_t)
    r.pcl_max, r.tau, r.mu, r.lambda_, r.eps = pcl_max, tau, mu, lam, eps
    r.softmax_scale, r.min_support, r.flags = softmax_scale, min_support, (DAM_RULE_GATHER_COLUMNS if gather_columns else 0)
    r.transform = TRANSFORMS[transform]
    return r


def dam_version() -> int:
    return int(lib().dam_version())


def dam_status_string(code: int) -> str:
    return lib().dam_status_string(code).decode()


def dam_mask_sizes(shape: Shape, rule: Optional[dam_rule_t], causal: bool = True):
    m, b, a = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    rc = lib().dam_mask_sizes(shape.ref, ctypes.byref(rule) if rule is not None else None, int(causal),
                              ctypes.byref(m), ctypes.byref(b), ctypes.byref(a))
    _check(rc, "dam_mask_sizes")
    return m.value, b.value, a.value


def _alloc(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(256, nbytes), dtype=torch.uint8, device=device)


def dam_build_masks(Q: torch.Tensor, K: torch.Tensor, shape: Shape, rule: dam_rule_t, mask: Optional[torch.Tensor] = None,
                    scratch: Optional[torch.Tensor] = None, scores_dump: Optional[torch.Tensor] = None):
    """Enqueues stage 1 on the current stream.  Returns (mask blob, scratch)."""
    if mask is None or scratch is None:
        mb, sb, _ = dam_mask_sizes(shape, rule)
        mask = mask if mask is not None else _alloc(mb, Q.device)
        scratch = scratch if scratch is not None else _alloc(sb, Q.device)
    rc = lib().dam_build_masks(_ptr(Q), _ptr(K), shape.ref, ctypes.byref(rule), _ptr(mask),
                               ctypes.c_size_t(mask.numel()), _ptr(scratch), ctypes.c_size_t(scratch.numel()),
                               _ptr(scores_dump), _stream(Q.device))
    _check(rc, "dam_build_masks")
    return mask, scratch


def dam_build_masks_static(Q: torch.Tensor, K: torch.Tensor, shape: Shape, rule: dam_rule_t, mask: torch.Tensor):
    """Stage 1 with the library's built-in scratch: for callers that cannot allocate device memory.
    `mask` must already exist (size from dam_mask_sizes); nothing is allocated here or in the library."""
    rc = lib().dam_build_masks_static(_ptr(Q), _ptr(K), shape.ref, ctypes.byref(rule), _ptr(mask),
                                      ctypes.c_size_t(mask.numel()), _stream(Q.device))
    _check(rc, "dam_build_masks_static")
    return mask


def dam_static_scratch_bytes() -> int:
    return int(lib().dam_static_scratch_bytes())


def dam_build_masks_from_scores(P: torch.Tensor, shape: Shape, rule: dam_rule_t, mask: Optional[torch.Tensor] = None,
                                scratch: Optional[torch.Tensor] = None):
    if mask is None or scratch is None:
        mb, sb, _ = dam_mask_sizes(shape, rule)
        mask = mask if mask is not None else _alloc(mb, P.device)
        scratch = scratch if scratch is not None else _alloc(sb, P.device)
    rc = lib().dam_build_masks_from_scores(_ptr(P), shape.ref, ctypes.byref(rule), _ptr(mask),
                                           ctypes.c_size_t(mask.numel()), _ptr(scratch),
                                           ctypes.c_size_t(scratch.numel()), _stream(P.device))
    _check(rc, "dam_build_masks_from_scores")
    return mask, scratch


def dam_mask_all_ones(shape: Shape, causal: bool, device, mask: Optional[torch.Tensor] = None) -> torch.Tensor:
    if mask is None:
        mb, _, _ = dam_mask_sizes(shape, None, causal)
        mask = _alloc(mb, device)
    rc = lib().dam_mask_all_ones(shape.ref, int(causal), _ptr(mask), ctypes.c_size_t(mask.numel()), _stream(device))
    _check(rc, "dam_mask_all_ones")
    return mask


def dam_sparse_attention(Q, K, V, mask, shape: Shape, causal: bool = True, softmax_scale: float = 0.0,
                         O: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                         scratch: Optional[torch.Tensor] = None):
    """Enqueues stage 2 on the current stream.  Returns (O, LSE [Hq, T] fp32, scratch)."""
    if O is None:
        O = torch.empty_like(Q)
    if lse is None:
        lse = torch.empty(shape.c.num_q_heads, shape.c.total_tokens, dtype=torch.float32, device=Q.device)
    if scratch is None:
        # a blob with gathered-column tiles records the scratch size it needs in its header
        off = _HDR.fields["attn_scratch_bytes"][1]
        need = int(mask[off: off + 8].cpu().numpy().view(np.uint64)[0]) if mask.numel() >= 256 else 256
        scratch = _alloc(max(256, need), Q.device)
    rc = lib().dam_sparse_attention(_ptr(Q), _ptr(K), _ptr(V), _ptr(mask), shape.ref, int(causal),
                                    shape.c.num_q_heads // shape.c.num_kv_heads, ctypes.c_float(softmax_scale),
                                    _ptr(O), _ptr(lse), _ptr(scratch), ctypes.c_size_t(scratch.numel()),
                                    _stream(Q.device))
    _check(rc, "dam_sparse_attention")
    return O, lse, scratch


def dam_capture_accumulate(P: torch.Tensor, shape: Shape, pcl_max: int, A: torch.Tensor, C: torch.Tensor):
    """A += the window maps of one batch of samples (P: the scores_dump of that batch), C += valid counts per row."""
    Hq = shape.c.num_q_heads
    assert A.dtype == torch.float32 and A.numel() == Hq * pcl_max * pcl_max and A.is_contiguous()
    assert C.dtype == torch.int32 and C.numel() == pcl_max
    assert P.dtype == torch.float32 and P.numel() == sum(Hq * min(S, pcl_max) ** 2 for S in shape.lengths)
    rc = lib().dam_capture_accumulate(_ptr(P), shape.ref, pcl_max, _ptr(A), _ptr(C), _stream(P.device))
    _check(rc, "dam_capture_accumulate")


def dam_capture_average(A: torch.Tensor, C: torch.Tensor, pcl_max: int, eps: float, shape: Shape) -> torch.Tensor:
    """Averaged maps for the sequences of `shape`, in the layout dam_build_masks_from_scores reads."""
    n = sum(shape.c.num_q_heads * min(S, pcl_max) ** 2 for S in shape.lengths)
    P = torch.empty(n, dtype=torch.float32, device=A.device)
    rc = lib().dam_capture_average(_ptr(A), _ptr(C), pcl_max, ctypes.c_float(eps), shape.ref, _ptr(P),
                                   _stream(A.device))
    _check(rc, "dam_capture_average")
    return P


def dam_sparse_attention_rows(Q, K, V, mask, shape: Shape, row_ranges, O: torch.Tensor, lse: torch.Tensor,
                              causal: bool = True, softmax_scale: float = 0.0,
                              scratch: Optional[torch.Tensor] = None):
    """Chunked prefill: stage 2 for the query rows [begin, end) of every sequence (row_ranges: [(begin, end)] per
    sequence).  O and LSE are updated in place on those rows only.  Returns scratch."""
    flat = [int(x) for pair in row_ranges for x in pair]
    assert len(flat) == 2 * shape.c.num_seqs
    host = (ctypes.c_int32 * len(flat))(*flat)
    dev = torch.tensor(flat, dtype=torch.int32, device=Q.device)
    if scratch is None:
        off = _HDR.fields["attn_scratch_bytes"][1]
        need = int(mask[off: off + 8].cpu().numpy().view(np.uint64)[0]) if mask.numel() >= 256 else 256
        scratch = _alloc(max(256, need), Q.device)
    rc = lib().dam_sparse_attention_rows(_ptr(Q), _ptr(K), _ptr(V), _ptr(mask), shape.ref, int(causal),
                                         shape.c.num_q_heads // shape.c.num_kv_heads, ctypes.c_float(softmax_scale),
                                         _ptr(O), _ptr(lse), host, _ptr(dev), _ptr(scratch),
                                         ctypes.c_size_t(scratch.numel()), _stream(Q.device))
    _check(rc, "dam_sparse_attention_rows")
    return scratch


def dam_decode_attention(q, K, V, mask, shape: Shape, positions: torch.Tensor, softmax_scale: float = 0.0,
                         O: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                         scratch: Optional[torch.Tensor] = None):
    """One new token per sequence against the KV cache `shape` describes (q, O: [B, Hq, d]; positions int32 [B]).

    Returns (O, LSE [B, Hq] fp32, scratch)."""
    B, Hq = shape.c.num_seqs, shape.c.num_q_heads
    assert q.is_contiguous() and tuple(q.shape) == (B, Hq, shape.c.head_dim)
    assert positions.dtype == torch.int32 and positions.numel() == B and positions.is_contiguous()
    if O is None:
        O = torch.empty_like(q)
    if lse is None:
        lse = torch.empty(B, Hq, dtype=torch.float32, device=q.device)
    if scratch is None:
        scratch = _alloc(256, q.device)
    rc = lib().dam_decode_attention(_ptr(q), _ptr(K), _ptr(V), _ptr(mask), shape.ref, _ptr(positions),
                                    Hq // shape.c.num_kv_heads, ctypes.c_float(softmax_scale), _ptr(O), _ptr(lse),
                                    _ptr(scratch), ctypes.c_size_t(scratch.numel()), _stream(q.device))
    _check(rc, "dam_decode_attention")
    return O, lse, scratch


def dam_mask_stats(mask: torch.Tensor, shape: Shape, active_elements: bool = False) -> dict:
    """Counts of a mask blob; with active_elements=True also the active cells per (sequence, head), counted by
    the library on the device (int64 tensor [num_seqs, num_q_heads], key "active_elements")."""
    out = (ctypes.c_uint64 * 5)()
    ae = torch.zeros(shape.c.num_seqs, shape.c.num_q_heads, dtype=torch.int64, device=mask.device) if active_elements else None
    rc = lib().dam_mask_stats(_ptr(mask), shape.ref, out, _ptr(ae), _stream(mask.device))
    _check(rc, "dam_mask_stats")
    st = {"tiles": int(out[0]), "full_tiles": int(out[1]), "causal_tiles": int(out[2]), "bytes_used": int(out[3]),
          "mask_tiles": int(out[4])}
    if active_elements:
        st["active_elements"] = ae
    return st


def dam_selftest_device_table(ordinals):
    """Runs the library's per-device table on a private table with a fake device query (no device needed).
    Returns (status code, sm_counts, (queries, set-up steps))."""
    n = len(ordinals)
    arr = (ctypes.c_int32 * max(1, n))(*ordinals)
    sm = (ctypes.c_int32 * max(1, n))()
    cnt = (ctypes.c_int32 * 2)()
    rc = lib().dam_selftest_device_table(arr, n, sm, cnt)
    return int(rc), [int(x) for x in sm[:n]], (int(cnt[0]), int(cnt[1]))


def dam_mask_expand_rows(mask: torch.Tensor, shape: Shape, seq: int, head: int, row_begin: int, nrows: int,
                         causal: bool = True) -> torch.Tensor:
    S = shape.lengths[seq]
    words = ((S + 127) // 128) * 4
    out = torch.empty(nrows, words, dtype=torch.int32, device=mask.device)
    rc = lib().dam_mask_expand_rows(_ptr(mask), shape.ref, seq, head, row_begin, nrows, int(causal), _ptr(out),
                                    _stream(mask.device))
    _check(rc, "dam_mask_expand_rows")
    return out


def attention_ran_on_tensor_cores(scratch: torch.Tensor) -> bool:
    """Test hook: word 4 of the attention scratch block says whether the tcgen05 kernel served the last call."""
    return int(scratch[16:20].cpu().numpy().view(np.uint32)[0]) == 1


def dam_poll_status(buf: torch.Tensor) -> int:
    return int(lib().dam_poll_status(_ptr(buf), _stream(buf.device)))


def dam_selftest_bounded_wait(device, limit_us: int = 20000):
    """Runs the bounded-wait self-test; returns (status read back, nanoseconds waited)."""
    scr = torch.zeros(256, dtype=torch.uint8, device=device)
    rc = lib().dam_selftest_bounded_wait(_ptr(scr), ctypes.c_size_t(256), ctypes.c_uint32(limit_us), _stream(device))
    _check(rc, "dam_selftest_bounded_wait")
    status = dam_poll_status(scr)
    waited = int(scr[8:16].cpu().numpy().view(np.uint64)[0])
    return status, waited


def dam_prefill_host(Qh: torch.Tensor, Kh: torch.Tensor, Vh: torch.Tensor, shape: Shape, rule: dam_rule_t,
                     Oh: torch.Tensor, lse_h: torch.Tensor, workspace: Optional[torch.Tensor], device,
                     causal: bool = True):
    """Host buffers in, host buffers out (copies inside the call).  workspace=None returns the size."""
    n = ctypes.c_size_t(0 if workspace is None else workspace.numel())
    rc = lib().dam_prefill_host(_ptr(Qh), _ptr(Kh), _ptr(Vh), shape.ref, ctypes.byref(rule), int(causal),
                                _ptr(Oh), _ptr(lse_h), _ptr(workspace), ctypes.byref(n), _stream(device))
    _check(rc, "dam_prefill_host")
    return n.value


# ----------------------------------------------------------------------------------------------
# Blob reader (host side, for tests and statistics): unpacks the sections of a mask blob.
# ----------------------------------------------------------------------------------------------
_HDR = np.dtype([("magic", "<u4"), ("status", "<u4"), ("version", "<u4"), ("flags", "<u4"),
                 ("num_seqs", "<i4"), ("num_q_heads", "<i4"), ("total_qblocks", "<i4"), ("rows", "<i4"),
                 ("tile_capacity", "<u4"), ("total_tiles", "<u4"), ("full_tiles", "<u4"), ("pcl_max", "<u4"),
                 ("off_seq", "<u8"), ("off_qbseq", "<u8"), ("off_dv", "<u8"), ("off_true", "<u8"),
                 ("off_tile_ptr", "<u8"), ("off_work", "<u8"), ("off_tiles", "<u8"), ("bytes_used", "<u8"),
                 ("causal_tiles", "<u8"), ("off_pairtab", "<u8"), ("total_pairs", "<i4"), ("prows", "<i4"),
                 ("gath_tiles", "<u8"), ("attn_scratch_bytes", "<u8"), ("mask_tiles", "<u8"), ("head_tile_cap", "<u8"), ("reserved", "<u8", (11,))])
_SEQ = np.dtype([("tok_start", "<i4"), ("S", "<i4"), ("L", "<i4"), ("nq", "<i4"), ("first_qblock", "<i4"),
                 ("W", "<i4"), ("nL", "<i4"), ("first_pair", "<i4"), ("dv_off", "<u8"), ("true_off", "<u8"),
                 ("p_off", "<u8"), ("cnt_off", "<u8"), ("gath_off", "<u8"), ("tile_base", "<u8")])


_ITEM = np.dtype([("head", "<i4"), ("tok0", "<i4"), ("qb0", "<i4"), ("S", "<i4"), ("a0", "<u4"), ("a1", "<u4"),
                  ("b1", "<u4"), ("seq_hasB", "<u4")])


def _unpack_bits(words: np.ndarray, n: int) -> np.ndarray:
    """uint32 words [..., W] -> uint8 bits [..., n] (bit j % 32 of word j / 32)."""
    b = np.unpackbits(words.astype("<u4").view(np.uint8), axis=-1, bitorder="little")
    return b[..., :n]


class MaskBlob:
    """Host copy of a mask blob with accessors for its sections."""

    def __init__(self, blob: torch.Tensor):
        hdr_bytes = blob[:256].cpu().numpy()
        self.hdr = np.frombuffer(hdr_bytes.tobytes(), dtype=_HDR)[0]
        assert self.hdr["magic"] == 0x4B4D4144, "not a DAM mask blob"
        used = int(max(self.hdr["bytes_used"], self.hdr["off_tiles"]))
        self.raw = blob[:used].cpu().numpy().tobytes()
        B = int(self.hdr["num_seqs"])
        self.seqs = np.frombuffer(self.raw, dtype=_SEQ, count=B, offset=int(self.hdr["off_seq"]))
        rows = int(self.hdr["rows"])
        self.tile_ptr = np.frombuffer(self.raw, dtype="<u4", count=rows + 1, offset=int(self.hdr["off_tile_ptr"]))
        self.items = np.frombuffer(self.raw, dtype=_ITEM, count=int(self.hdr["prows"]),
                                   offset=int(self.hdr["off_work"]))
        self.pair_tab = np.frombuffer(self.raw, dtype="<u4", count=int(self.hdr["total_pairs"]),
                                      offset=int(self.hdr["off_pairtab"]))
        # every row owns a fixed range of tiles[]: its entries, then possibly zero entries (kind 0) as padding
        self.tiles = np.frombuffer(self.raw, dtype="<u4", count=int(self.tile_ptr[rows]),
                                   offset=int(self.hdr["off_tiles"]))

    @property
    def scored_on_tensor_cores(self) -> bool:
        """Test hook: the window map of this blob was computed by the tcgen05 scoring kernel."""
        return int(self.hdr["reserved"][0]) == 1

    def pattern_bits(self, seq: int, head: int):
        """(D, Drev, V) as uint8 [L]."""
        s = self.seqs[seq]
        L, W = int(s["L"]), int(s["W"])
        off = int(self.hdr["off_dv"]) + 4 * (int(s["dv_off"]) + head * 3 * W)
        w = np.frombuffer(self.raw, dtype="<u4", count=3 * W, offset=off).reshape(3, W)
        bits = _unpack_bits(w, L)
        return bits[0], bits[1], bits[2]

    def true_mask(self, seq: int, head: int) -> np.ndarray:
        s = self.seqs[seq]
        L, W = int(s["L"]), int(s["W"])
        off = int(self.hdr["off_true"]) + 4 * (int(s["true_off"]) + head * L * W)
        w = np.frombuffer(self.raw, dtype="<u4", count=L * W, offset=off).reshape(L, W)
        return _unpack_bits(w, L)

    def row_tiles(self, seq: int, head: int, qb: int):
        """(kv tile indices, kinds) of query block qb of (seq, head)."""
        row = head * int(self.hdr["total_qblocks"]) + int(self.seqs[seq]["first_qblock"]) + qb
        e = self.row_entries(seq, head, qb)
        kinds = (e >> 28).astype(np.int64)
        idx = np.where(kinds == 3, e & 0xFFFF, e & 0x0FFFFFFF).astype(np.int64)
        return idx, kinds

    def row_entries(self, seq: int, head: int, qb: int) -> np.ndarray:
        row = head * int(self.hdr["total_qblocks"]) + int(self.seqs[seq]["first_qblock"]) + qb
        e = self.tiles[self.tile_ptr[row]: self.tile_ptr[row + 1]]
        return e[(e >> 28) != 0]                                    # without the padding
