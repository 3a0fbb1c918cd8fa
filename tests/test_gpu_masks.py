"""Stage-1 parity on the GPU, through the C ABI: masks must equal the oracle's bit for bit when both
start from the same fp32 score tensor."""
import numpy as np
import pytest
import torch

from oracle import dam_oracle as orc
from paper_2506_11104_b200 import binding as B
from paper_2506_11104_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _shape(w):
    return B.make_shape(w.cu_seqlens, w.num_q_heads, w.num_kv_heads, w.head_dim, w.Q.dtype, DEV)


def _rule(w, **kw):
    return B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps, **kw)


GATHER = [False, True]


def _band(L, wdt):
    i, j = np.indices((L, L))
    return ((i - j >= 0) & (i - j < wdt)).astype(np.float32)


def _from_scores_case(lengths, Hq, pcl, P_list, tau, mu, min_support=1):
    cu = np.concatenate([[0], np.cumsum(lengths)]).tolist()
    shape = B.make_shape(cu, Hq, Hq, 64, torch.float32, DEV)
    rule = B.make_rule(pcl, tau, mu, min_support=min_support)
    flat = np.concatenate([p.reshape(-1) for per in P_list for p in per]).astype(np.float32)
    blob, _ = B.dam_build_masks_from_scores(torch.from_numpy(flat).to(DEV), shape, rule)
    assert B.dam_poll_status(blob) == 0
    masks = [[orc.head_mask_from_probs(np.ascontiguousarray(P_list[b][h]), S, tau, mu, min_support=min_support)
              for h in range(Hq)] for b, S in enumerate(lengths)]
    n = H.check_blob_against_oracle(blob, shape, masks)
    return blob, shape, masks, n


def test_injected_band_sink_and_ties():
    """Closed-form score tensors: a band, a sink column, random lower-triangular noise, an exact tie."""
    L = 256
    rng = np.random.default_rng(0)
    sink = np.zeros((L, L), np.float32)
    sink[:, 0] = 1.0
    noise = np.tril(rng.random((L, L)) * 0.05).astype(np.float32)
    tie = np.zeros((L, L), np.float32)
    r, need = 56, int(np.ceil(0.8 * (L - 56)))
    for t in range(need):
        tie[r + t, t] = 1.0
    P = [[_band(L, 32), sink, noise, tie]]
    blob, shape, masks, n = _from_scores_case([1000], 4, L, P, 0.3, 0.8)
    assert n > 0
    assert np.flatnonzero(masks[0][0].V).tolist() == list(range(L - 40, L))     # last floor(32 / 0.8) columns
    assert masks[0][3].D[r] == 1


@pytest.mark.parametrize("lengths,pcl", [([300], 200), ([129, 1, 640, 77], 130), ([2048], 512), ([100], 256)])
def test_ragged_lengths_random_scores(lengths, pcl):
    """Windows and sequences that are not multiples of the tile or word size, several sequences, S <= L."""
    rng = np.random.default_rng(sum(lengths))
    Hq = 3
    P = []
    for S in lengths:
        L = min(S, pcl)
        per = []
        for h in range(Hq):
            p = np.tril(rng.random((L, L)) * 0.04).astype(np.float32)
            p += _band(L, 3 + 17 * h) * 0.5
            p[:, min(5, L - 1)] = 1.0
            per.append(np.tril(p).astype(np.float32))
        P.append(per)
    _from_scores_case(lengths, Hq, pcl, P, 0.3, 0.8)


def test_wide_band_gives_full_tiles_and_mu_extremes():
    L, S = 512, 2000
    P = [[_band(L, 400), _band(L, 400)]]
    blob, shape, masks, _ = _from_scores_case([S], 2, L, P, 0.3, 0.8)
    st = B.dam_mask_stats(blob, shape)
    assert st["full_tiles"] > 0 and st["tiles"] > st["full_tiles"]
    # mu <= 0: every pattern matches; mu > 1: none
    _from_scores_case([S], 2, L, P, 0.3, 0.0)
    b2, s2, m2, _ = _from_scores_case([S], 2, L, P, 0.3, 1.5)
    assert not m2[0][0].D.any()
    _from_scores_case([S], 2, L, P, 0.3, 0.8, min_support=50)


def test_threshold_boundary_values_bit_exact():
    """Score values packed around the flip point of the fp32 threshold chain, for several tau."""
    L = 128
    for tau in (0.3, 0.1, 0.05, 0.02):
        centre = np.float32((tau / 2 + 1e-4) ** 2)
        bits = centre.view(np.uint32).astype(np.int64) + np.arange(-L * L // 2, L * L // 2)
        P = np.tril(bits.astype(np.uint32).view(np.float32).reshape(L, L)).astype(np.float32)
        _from_scores_case([L], 1, L, [[P]], tau, 0.8)


def _build_and_check(w, qblocks=None, gather=False):
    shape, rule = _shape(w), _rule(w, gather_columns=gather)
    Q, K = w.Q.to(DEV), w.K.to(DEV)
    lengths = shape.lengths
    n = sum(w.num_q_heads * min(S, w.pcl_max) ** 2 for S in lengths)
    dump = torch.zeros(n, dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(Q, K, shape, rule, scores_dump=dump)
    assert B.dam_poll_status(blob) == 0
    masks = H.oracle_masks_from_dump(w, dump.cpu().numpy())
    # bf16 with head_dim 128 or 64 is scored by the tcgen05 kernel, everything else by the CUDA-core kernel
    assert B.MaskBlob(blob).scored_on_tensor_cores == (w.Q.dtype == torch.bfloat16 and w.head_dim in (64, 128))
    H.check_blob_against_oracle(blob, shape, masks, qblocks_per_head=qblocks)
    # a second build without the dump gives the identical blob (dump does not change decisions; deterministic)
    blob2, _ = B.dam_build_masks(Q, K, shape, rule)
    used = B.dam_mask_stats(blob, shape)["bytes_used"]
    mb1, mb2 = B.MaskBlob(blob), B.MaskBlob(blob2)
    assert mb1.seqs.tobytes() == mb2.seqs.tobytes() and mb1.tile_ptr.tobytes() == mb2.tile_ptr.tobytes()
    assert mb1.tiles.tobytes() == mb2.tiles.tobytes() and used == int(mb2.hdr["bytes_used"])
    for b in range(len(lengths)):
        for h in range(0, w.num_q_heads, max(1, w.num_q_heads // 4)):
            assert all(np.array_equal(x, y) for x, y in zip(mb1.pattern_bits(b, h), mb2.pattern_bits(b, h)))
            assert np.array_equal(mb1.true_mask(b, h), mb2.true_mask(b, h))
    # work list: one item per (head, pair of adjacent query blocks), most listed tiles first
    tq = int(mb1.hdr["total_qblocks"])
    seen, keys = set(), []
    for it in mb1.items:
        b, has2 = int(it["seq_hasB"] & 0x7FFFFFFF), int(it["seq_hasB"] >> 31)
        sq = mb1.seqs[b]
        row = int(it["head"]) * tq + int(sq["first_qblock"]) + int(it["qb0"])
        assert int(it["qb0"]) % 2 == 0 and int(it["tok0"]) == int(sq["tok_start"]) and int(it["S"]) == int(sq["S"])
        assert has2 == (int(it["qb0"]) + 1 < int(sq["nq"]))
        # the pair's entries: block 2p from tile_ptr[row], block 2p+1 directly behind, then zero padding
        qb0 = int(it["qb0"])
        nA, nB = len(mb1.row_entries(b, int(it["head"]), qb0)), (len(mb1.row_entries(b, int(it["head"]), qb0 + 1)) if has2 else 0)
        assert int(it["a0"]) == int(mb1.tile_ptr[row]) and int(it["a1"]) == int(it["a0"]) + nA
        assert int(it["b1"]) == int(it["a1"]) + nB and int(it["b1"]) <= int(mb1.tile_ptr[row + 1 + has2])
        if has2:
            assert int(it["a1"]) == int(mb1.tile_ptr[row + 1])
        assert not mb1.tiles[int(it["b1"]): int(mb1.tile_ptr[row + 1 + has2])].any()
        seen.add((int(it["head"]), b, int(it["qb0"])))
        keys.append(int(it["b1"]) - int(it["a0"]))
    assert len(seen) == int(mb1.hdr["prows"]) == len(mb1.items)
    assert all(a >= c for a, c in zip(keys[:-1], keys[1:]))
    return blob, shape, masks, dump


def _score_closeness(w, dump, masks, heads):
    """GPU fp32 map vs the float64 map; every cell whose decision differs must sit within 2 % of p*."""
    Q, K, _ = H.host_qkv(w)
    P = H.split_dump(dump.cpu().numpy(), [b - a for a, b in zip(w.cu_seqlens[:-1], w.cu_seqlens[1:])],
                     w.num_q_heads, w.pcl_max)
    g = w.num_q_heads // w.num_kv_heads
    pstar = (w.tau / 2 + np.sqrt(w.eps)) ** 2
    flipped = total = 0
    for b in range(len(w.cu_seqlens) - 1):
        t0, t1 = w.cu_seqlens[b], w.cu_seqlens[b + 1]
        L = min(t1 - t0, w.pcl_max)
        for h in heads:
            P64 = orc.window_probs(Q[t0:t1, h], K[t0:t1, h // g], L, 1 / np.sqrt(w.head_dim))
            assert np.abs(P[b][h] - P64).max() < 2e-5
            M64 = orc.true_mask_f64(P64, w.tau, w.lam, w.eps)
            diff = M64 != masks[b][h].M
            flipped += int(diff.sum())
            total += L * (L + 1) // 2
            if diff.any():
                assert np.all(np.abs(P64[diff] - pstar) <= 0.02 * pstar)
    return flipped, total


def test_config0_full():
    w = synth.config0()
    blob, shape, masks, dump = _build_and_check(w)
    flipped, total = _score_closeness(w, dump, masks, range(w.num_q_heads))
    assert flipped <= 1e-3 * total
    # planted structure is recovered
    assert masks[0][0].V[0] == 1 and masks[0][0].D[:8].all()
    assert all(masks[0][1].V[p] for p in w.plans[0][1].stripes)


@pytest.mark.parametrize("lengths,pcl,Hq,Hkv,d,dtype", [
    ([700], 256, 4, 2, 128, torch.bfloat16),
    ([333, 1000, 64], 200, 4, 1, 64, torch.bfloat16),
    ([513], 300, 2, 2, 32, torch.float32),
    ([2100, 700], 384, 8, 2, 64, torch.bfloat16),
])
@pytest.mark.parametrize("gather", GATHER)
def test_small_cases_scored_on_gpu(lengths, pcl, Hq, Hkv, d, dtype, gather):
    w = synth.small_case(0, Hq, Hkv, d, pcl, seed=len(lengths), dtype=dtype, lengths=lengths)
    blob, shape, masks, dump = _build_and_check(w, gather=gather)
    flipped, total = _score_closeness(w, dump, masks, range(Hq))
    assert flipped <= 2e-3 * total


@pytest.mark.parametrize("gather", GATHER)
def test_config1_full_size_masks(gather):
    """Llama-3-8B-shaped layer, 8192 tokens, PCL 1024: every head's D, V and true mask, sampled q-blocks."""
    w = synth.config1()
    blob, shape, masks, dump = _build_and_check(w, qblocks=12, gather=gather)
    flipped, total = _score_closeness(w, dump, masks, [0, 9, 31])
    assert flipped <= 1e-3 * total
    st = B.dam_mask_stats(blob, shape)
    assert (0.02 if gather else 0.03) <= st["tiles"] / st["causal_tiles"] <= 0.45


def test_config2_layer_masks():
    """A layer of the 32-layer stack: 32768 tokens, PCL 2048."""
    w = synth.config2_layer(3, DEV)
    blob, shape, masks, dump = _build_and_check(w, qblocks=10, gather=True)
    st = B.dam_mask_stats(blob, shape)
    assert 0.01 <= st["tiles"] / st["causal_tiles"] <= 0.30
    # the scoring kernel's own map at PCL 2048 (16 kv tiles per query block, all four softmax groups and their
    # merge) against the float64 map
    flipped, total = _score_closeness(w, dump, masks, [2, 11, 20, 29])
    print(f"config 2: {flipped} of {total} window cells decided differently from the float64 map")
    assert flipped <= 1e-3 * total


@pytest.mark.parametrize("gather", GATHER)
def test_config4_varlen_masks(gather):
    w = synth.config4(lengths=(4096, 16384, 32768, 65536))
    blob, shape, masks, dump = _build_and_check(w, qblocks=8, gather=gather)
    flipped, total = _score_closeness(w, dump, masks, [1, 14, 30])          # every sequence, three heads
    print(f"config 4: {flipped} of {total} window cells decided differently from the float64 map")
    assert flipped <= 1e-3 * total


def test_config3_shape_masks():
    """131072 tokens, PCL 4096 (config 3): all heads' pattern bits and true masks, sampled q-blocks."""
    w = synth.config3(device=DEV)
    blob, shape, masks, dump = _build_and_check(w, qblocks=8)
    st = B.dam_mask_stats(blob, shape)
    assert 0.005 <= st["tiles"] / st["causal_tiles"] <= 0.08
    # PCL 4096: a query block sweeps up to 32 kv tiles; the map itself against the float64 map
    flipped, total = _score_closeness(w, dump, masks, [0, 13, 26])
    print(f"config 3: {flipped} of {total} window cells decided differently from the float64 map")
    assert flipped <= 1e-3 * total


def test_mask_tile_count_is_independent_of_gathering():
    """The 128 x 128 tiles of the mask with an active cell are counted the same whether matched columns are
    listed as vertical tiles or served by gathered-column tiles; the executed tile list shrinks."""
    w = synth.config1()
    shape = _shape(w)
    Q, K = w.Q.to(DEV), w.K.to(DEV)
    plain, _ = B.dam_build_masks(Q, K, shape, _rule(w))
    gath, _ = B.dam_build_masks(Q, K, shape, _rule(w, gather_columns=True))
    a, b = B.dam_mask_stats(plain, shape), B.dam_mask_stats(gath, shape)
    assert a["mask_tiles"] == a["tiles"] == b["mask_tiles"]
    assert b["tiles"] < a["tiles"]


@pytest.mark.parametrize("lengths,pcl,gather", [
    ([1], 64, False), ([127, 128, 129], 128, True), ([700, 260, 5], 96, True), ([2100], 512, True),
    ([2100], 512, False), ([640, 64], 1024, True),
])
def test_tile_lists_sit_at_fixed_places(lengths, pcl, gather):
    """Every pair of adjacent query blocks owns the range of tiles[] that its rows' upper bounds add up to: the
    ranges follow from the shapes alone, tile the whole capacity, and hold the two rows' entries back to back
    followed by zero entries only."""
    Hq, Hkv, d = 4, 2, 128
    w = synth.small_case(0, Hq, Hkv, d, pcl, seed=13, dtype=torch.bfloat16, lengths=lengths)
    shape = B.make_shape(w.cu_seqlens, Hq, Hkv, d, torch.bfloat16, DEV)
    rule = B.make_rule(w.pcl_max, w.tau, w.mu, w.lam, w.eps, gather_columns=gather)
    blob, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule)
    assert B.dam_poll_status(blob) == 0
    mb = B.MaskBlob(blob)
    hdr, tq = mb.hdr, int(mb.hdr["total_qblocks"])

    def bound(qb, nL, L):                      # upper bound on the listed tiles of a query block (host restatement)
        gf = (2 * L - 1 + 127) // 128
        if gather and L > 0 and qb >= gf:
            return nL + min(qb + 1, nL + 1)
        return min(qb + 1, 2 * nL + 1)

    cap_head = int(hdr["head_tile_cap"])
    assert int(hdr["tile_capacity"]) == Hq * cap_head == int(mb.tile_ptr[-1])
    assert int(hdr["bytes_used"]) == int(hdr["off_tiles"]) + 4 * Hq * cap_head
    listed = 0
    for h in range(Hq):
        at = h * cap_head
        for b, sq in enumerate(mb.seqs):
            nq, nL, L = int(sq["nq"]), int(sq["nL"]), int(sq["L"])
            assert at == h * cap_head + int(sq["tile_base"])
            for qb0 in range(0, nq, 2):
                row = h * tq + int(sq["first_qblock"]) + qb0
                nblk = 2 if qb0 + 1 < nq else 1
                end = at + sum(bound(qb0 + x, nL, L) for x in range(nblk))
                assert int(mb.tile_ptr[row]) == at
                nA = len(mb.row_entries(b, h, qb0))
                nB = len(mb.row_entries(b, h, qb0 + 1)) if nblk == 2 else 0
                if nblk == 2:
                    assert int(mb.tile_ptr[row + 1]) == at + nA
                seg = mb.tiles[at:end]
                assert ((seg[:nA + nB] >> 28) != 0).all() and not seg[nA + nB:].any()
                listed += nA + nB
                at = end
        assert at == (h + 1) * cap_head
    assert listed == int(hdr["total_tiles"])


def test_multi_sample_capture_masks_bit_exact():
    """Three batches of samples of mixed lengths are accumulated on the GPU; the masks built from the averaged
    maps equal, bit for bit, the oracle's masks from its own fp32 average of the same per-sample score tensors."""
    Hq, Hkv, d, pcl = 4, 2, 64, 160
    batches = [[400, 100], [160, 300, 37], [512]]
    A = torch.zeros(Hq * pcl * pcl, dtype=torch.float32, device=DEV)
    C = torch.zeros(pcl, dtype=torch.int32, device=DEV)
    per_head = [[] for _ in range(Hq)]
    w_last = None
    for k, lengths in enumerate(batches):
        w = synth.small_case(0, Hq, Hkv, d, pcl, seed=30 + k, dtype=torch.bfloat16, lengths=lengths)
        shape = B.make_shape(w.cu_seqlens, Hq, Hkv, d, w.Q.dtype, DEV)
        rule = B.make_rule(pcl, w.tau, w.mu, w.lam, w.eps)
        n = sum(Hq * min(S, pcl) ** 2 for S in lengths)
        dump = torch.zeros(n, dtype=torch.float32, device=DEV)
        B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule, scores_dump=dump)
        B.dam_capture_accumulate(dump, shape, pcl, A, C)
        P = H.split_dump(dump.cpu().numpy(), lengths, Hq, pcl)
        for b in range(len(lengths)):
            for h in range(Hq):
                per_head[h].append(P[b][h])
        w_last = w
    # masks for new inputs (one longer than the window, one shorter) from the averaged maps
    target = [700, 90]
    tshape = B.make_shape([0, 700, 790], Hq, Hkv, d, torch.bfloat16, DEV)
    rule = B.make_rule(pcl, w_last.tau, w_last.mu, w_last.lam, w_last.eps)
    Pavg = B.dam_capture_average(A, C, pcl, w_last.eps, tshape)
    blob, _ = B.dam_build_masks_from_scores(Pavg, tshape, rule)
    assert B.dam_poll_status(blob) == 0
    want_C = [sum(1 for ls in batches for S in ls if min(S, pcl) > i) for i in range(pcl)]
    assert C.cpu().tolist() == want_C
    masks = []
    for S in target:
        L = min(S, pcl)
        row = []
        for h in range(Hq):
            Abar, _ = orc.capture_average(per_head[h], pcl, w_last.eps, dtype=np.float32)
            row.append(orc.head_mask_from_probs(np.ascontiguousarray(Abar[:L, :L]), S, w_last.tau, w_last.mu,
                                                w_last.lam, w_last.eps))
        masks.append(row)
    H.check_blob_against_oracle(blob, tshape, masks)


@pytest.mark.parametrize("transform,lam,tau", [
    ("log", 0.0, 13.0), ("sqrt", 0.0, 0.1), ("arcsinh", 0.0, 0.01), ("average", 0.0, 0.01),
    ("boxcox", 0.25, 1.5), ("boxcox", 0.0, 13.0), ("yeo_johnson", 0.5, 0.01), ("yeo_johnson", 0.0, 0.01),
    ("zscore", 0.0, 1.0), ("minmax", 0.0, 0.02), ("sum", 0.0, 0.03),
])
def test_other_amplifications_bit_exact_from_scores(transform, lam, tau):
    """The Appendix-B amplifications through the C ABI: the same fp32 score tensor on both sides, masks bit-exact
    (true mask, D, V and the tile lists of sampled query blocks)."""
    w = synth.small_case(0, 4, 2, 64, 160, seed=40, dtype=torch.bfloat16, lengths=[500, 120])
    shape = B.make_shape(w.cu_seqlens, 4, 2, 64, w.Q.dtype, DEV)
    n = sum(4 * min(S, 160) ** 2 for S in shape.lengths)
    dump = torch.zeros(n, dtype=torch.float32, device=DEV)
    B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, B.make_rule(160, w.tau, w.mu), scores_dump=dump)
    rule = B.make_rule(160, tau, w.mu, lam, w.eps, transform=transform)
    if transform == "sum":
        # the raw sum of three inputs' maps (here three times the same map), handed in as it is
        dump = dump * 3.0
        blob, _ = B.dam_build_masks_from_scores(dump, shape, rule)
        blob2 = blob
    elif transform in ("zscore", "minmax"):
        blob, _ = B.dam_build_masks_from_scores(dump, shape, rule)
        # thresholds that depend on the finished map: the scoring path takes them when it gets a buffer for the map
        with pytest.raises(B.DamError):
            B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule)
        dump2 = torch.zeros_like(dump)
        blob2, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule, scores_dump=dump2)
        assert torch.equal(dump2, dump)
    else:
        blob, _ = B.dam_build_masks_from_scores(dump, shape, rule)
        # and the fused scoring path decides on the same values
        blob2, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule)
    assert B.dam_poll_status(blob) == 0 and B.dam_poll_status(blob2) == 0
    P = H.split_dump(dump.cpu().numpy(), shape.lengths, 4, 160)
    masks = [[orc.head_mask_from_probs(np.ascontiguousarray(P[b][h]), S, tau, w.mu, lam, w.eps, method=transform)
              for h in range(4)] for b, S in enumerate(shape.lengths)]
    active = sum(int(m.M.sum()) for row in masks for m in row)
    assert active > 0
    H.check_blob_against_oracle(blob, shape, masks)
    H.check_blob_against_oracle(blob2, shape, masks)


def test_active_element_count_matches_the_extended_mask():
    """dam_mask_stats' per-(sequence, head) active-cell counts (a kernel of the library working on the pattern
    bits) against the sum of the oracle's extended-mask rows, with and without gathered-column tile lists."""
    w = synth.small_case(0, 4, 2, 64, 96, seed=50, dtype=torch.bfloat16, lengths=[400, 150, 60, 96, 191])
    shape = B.make_shape(w.cu_seqlens, 4, 2, 64, w.Q.dtype, DEV)
    rule = B.make_rule(96, w.tau, w.mu)
    n = sum(4 * min(S, 96) ** 2 for S in shape.lengths)
    dump = torch.zeros(n, dtype=torch.float32, device=DEV)
    blob, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule, scores_dump=dump)
    masks = H.oracle_masks_from_dump(w, dump.cpu().numpy())
    got = B.dam_mask_stats(blob, shape, active_elements=True)["active_elements"].cpu().numpy()
    for b, S in enumerate(shape.lengths):
        for h in range(4):
            assert int(got[b, h]) == int(masks[b][h].rows(list(range(S))).sum()), (b, h)
    # an all-ones blob has no pattern sections to count from
    with pytest.raises(B.DamError):
        B.dam_mask_stats(B.dam_mask_all_ones(shape, True, DEV), shape, active_elements=True)


def _per_head_tile_density(w):
    shape, rule = _shape(w), _rule(w)
    blob, _ = B.dam_build_masks(w.Q.to(DEV), w.K.to(DEV), shape, rule)
    mb = B.MaskBlob(blob)
    Hq, cap = int(mb.hdr["num_q_heads"]), int(mb.hdr["head_tile_cap"])
    listed = (mb.tiles.reshape(Hq, cap) != 0).sum(axis=1)
    return listed / (int(mb.hdr["causal_tiles"]) / Hq)


def test_per_head_densities_are_heterogeneous():
    """The planted-pattern draw gives per-head tile densities (tiles with an active cell over causal tiles) that
    span what the configurations ask for: a few per cent to about 40 % over the heads of the 8192-token layer, about
    1 % to the cap the threshold allows (a row keeps at most 1 / p* = 1587 keys at tau 0.05, so a band is at most a
    dozen tiles wide next to the 16 column tiles of the window) over the heads of the 32-layer stack."""
    d1 = _per_head_tile_density(synth.config1(DEV))
    assert d1.min() <= 0.06 and d1.max() >= 0.33 and 0.15 <= np.median(d1) <= 0.33, (d1.min(), np.median(d1), d1.max())
    d2 = np.concatenate([_per_head_tile_density(synth.config2_layer(l, DEV)) for l in (2, 3, 4, 5)])
    assert d2.min() <= 0.025 and d2.max() >= 0.15 and d2.max() <= 0.30, (d2.min(), d2.max())
    # heads of one layer differ by a large factor, which is what the longest-first work list has to balance
    assert d2.max() / d2.min() >= 6
