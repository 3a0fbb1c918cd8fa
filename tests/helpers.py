"""Shared helpers for the parity tests: run the oracle on the same arrays the CUDA library saw."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dam_oracle as orc

TILE = 128


def to_f32_numpy(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def host_qkv(w):
    """float32 numpy copies of a workload's Q, K, V, converted once and kept on the workload object."""
    if not hasattr(w, "_host_qkv"):
        w._host_qkv = tuple(to_f32_numpy(x) for x in (w.Q, w.K, w.V))
    return w._host_qkv


def split_dump(dump: np.ndarray, lengths, Hq: int, pcl: int):
    """Flat fp32 score dump -> P[seq][head] arrays of shape [L, L]."""
    out, off = [], 0
    for S in lengths:
        L = min(S, pcl)
        per = []
        for h in range(Hq):
            per.append(dump[off: off + L * L].reshape(L, L))
            off += L * L
        out.append(per)
    return out


def oracle_masks_from_dump(w, dump: np.ndarray, min_support: int = 1, heads=None):
    lengths = [b - a for a, b in zip(w.cu_seqlens[:-1], w.cu_seqlens[1:])]
    P = split_dump(dump, lengths, w.num_q_heads, w.pcl_max)
    out = []
    for b, S in enumerate(lengths):
        out.append([orc.head_mask_from_probs(np.ascontiguousarray(P[b][h]), S, w.tau, w.mu, w.lam, w.eps, min_support)
                    if (heads is None or h in heads) else None for h in range(w.num_q_heads)])
    return out


def nonempty_tiles(rows_bits: np.ndarray, S: int):
    """rows_bits uint8 [n, S] for the rows of one q-block -> (sorted kv tile indices with any bit, full flags)."""
    nk = (S + TILE - 1) // TILE
    pad = np.zeros((rows_bits.shape[0], nk * TILE), np.uint8)
    pad[:, :S] = rows_bits
    t = pad.reshape(rows_bits.shape[0], nk, TILE)
    anyb = t.any(axis=(0, 2))
    full = (t.sum(axis=(0, 2)) == TILE * TILE) if rows_bits.shape[0] == TILE else np.zeros(nk, bool)
    return np.flatnonzero(anyb), full


def check_blob_against_oracle(blob, shape, masks, qblocks_per_head=None, rng=None, lib=None):
    """Bit-exact comparison of a mask blob with the oracle's (M, D, V) and extension rule.

    For every (seq, head): D, V, true mask equal; for the chosen q-blocks: the tile list equals the set
    of tiles that hold at least one active cell of the oracle's S x S mask, FULL tiles are all ones, and
    the rows expanded by the library (dam_mask_expand_rows) equal the oracle's rows cell by cell."""
    from paper_2506_11104_b200 import binding as B
    mb = B.MaskBlob(blob)
    rng = rng or np.random.default_rng(0)
    Hq = shape.c.num_q_heads
    n_tiles_checked = 0
    for b, S in enumerate(shape.lengths):
        if S == 0:
            continue
        for h in range(Hq):
            hm = masks[b][h]
            if hm is None:
                continue
            D, Drev, V = mb.pattern_bits(b, h)
            assert np.array_equal(D, hm.D), f"D differs seq {b} head {h}"
            assert np.array_equal(V, hm.V), f"V differs seq {b} head {h}"
            assert np.array_equal(Drev, hm.D[::-1]), f"Drev differs seq {b} head {h}"
            assert np.array_equal(mb.true_mask(b, h), hm.M), f"true mask differs seq {b} head {h}"
            nq = (S + TILE - 1) // TILE
            if qblocks_per_head is None or nq <= qblocks_per_head:
                qbs = list(range(nq))
            else:
                L = hm.L
                special = {0, nq - 1, (L - 1) // TILE, min(nq - 1, L // TILE), min(nq - 1, (2 * L - 1) // TILE),
                           min(nq - 1, (2 * L - 1) // TILE + 1)}
                extra = rng.choice(nq, size=max(0, qblocks_per_head - len(special)), replace=False)
                qbs = sorted(special | set(int(x) for x in extra))
            gather = bool(int(mb.hdr["flags"]) & 4)
            L = hm.L
            g_first = (2 * L - 1 + TILE - 1) // TILE if (gather and L > 0) else 1 << 30
            nV = int(hm.V.sum())
            for qb in qbs:
                i0, i1 = qb * TILE, min(S, qb * TILE + TILE)
                rows = hm.rows(list(range(i0, i1)))
                kbs, kinds = mb.row_tiles(b, h, qb)
                if qb >= g_first:
                    # gathered-column tiles first: ceil(nV / 128) of them, holding the matched columns in order
                    ng = (nV + TILE - 1) // TILE
                    ent = mb.row_entries(b, h, qb)
                    assert np.array_equal(kinds[:ng], np.full(ng, 3)) and np.array_equal(kbs[:ng], np.arange(ng))
                    assert all(int((e >> 16) & 0xFF) + 1 == min(TILE, nV - g * TILE) for g, e in enumerate(ent[:ng]))
                    band = rows.copy()
                    band[:, :L][:, hm.V.astype(bool)] = 0          # columns served by the gathered tiles
                    want, full = nonempty_tiles(band, S)
                    kbs, kinds = kbs[ng:], kinds[ng:]
                else:
                    want, full = nonempty_tiles(rows, S)
                assert np.array_equal(kbs, want), f"tile list differs seq {b} head {h} qb {qb}: {kbs} vs {want}"
                for kb, kind in zip(kbs, kinds):
                    assert kind in (1, 2)
                    if kind == 1:
                        assert full[kb], f"tile ({qb},{kb}) listed FULL but is not all ones"
                n_tiles_checked += len(kbs)
                got = B.dam_mask_expand_rows(blob, shape, b, h, i0, i1 - i0, causal=True).cpu().numpy()
                gotbits = np.unpackbits(got.astype("<u4").view(np.uint8), axis=-1, bitorder="little")[:, :S]
                assert np.array_equal(gotbits, rows), f"expanded rows differ seq {b} head {h} qb {qb}"
    return n_tiles_checked


def attention_errors(O_gpu: torch.Tensor, lse_gpu: torch.Tensor, w, masks, seq: int, head: int, rows, causal=True,
                     all_ones=False):
    """Max / mean abs error of O and max abs error of LSE on the given rows of (seq, head) vs the oracle."""
    Q, K, V = host_qkv(w)
    hm = None if all_ones else masks[seq][head]
    O_ref, lse_ref = orc.attention(Q, K, V, w.cu_seqlens, seq, head, rows, hm, causal=causal)
    t0 = w.cu_seqlens[seq]
    idx = torch.as_tensor(np.asarray(rows) + t0, device=O_gpu.device)
    O = O_gpu[idx, head, :].double().cpu().numpy()
    lse = lse_gpu[head, idx].double().cpu().numpy()
    err = np.abs(O - O_ref)
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), ~fin), "empty rows (LSE = -inf) differ"
    lse_err = np.abs(lse[fin] - lse_ref[fin]).max() if fin.any() else 0.0
    return float(err.max()), float(err.mean()), float(lse_err)
