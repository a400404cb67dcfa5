"""The C-ABI library loads without a GPU, exports what the header declares, and rejects
malformed requests before touching the device."""
import os
import re

import pytest

from paper_2609_28568_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def test_exports_match_header(L):
    header = open(os.path.join(ROOT, "include", "nb_linear.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(nb_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_version_and_out_elems(L):
    assert L.nb_version() == 100
    assert L.nb_linear_out_elems(128, 3072, binding.ACT_NONE) == 128 * 3072
    assert L.nb_linear_out_elems(128, 3072, binding.ACT_GELU) == 2 * 128 * 3072
    assert L.nb_linear_out_elems(16, 6144, binding.ACT_SWIGLU) == 16 * 3072 + 16 * 6144
    assert L.nb_linear_out_elems(16, 7, binding.ACT_SWIGLU) == -1
    assert L.nb_linear_out_elems(-1, 8, binding.ACT_NONE) == -1
    assert L.nb_linear_out_elems(1, 8, 9) == -1


def test_stream_is_per_thread_state(L):
    assert L.nb_get_stream() in (None, 0)
    L.nb_set_stream(0x1000)
    assert L.nb_get_stream() == 0x1000
    L.nb_set_stream(None)


def test_malformed_requests_are_rejected_without_a_device(L):
    P = 0x10000  # a fake, aligned device address: never dereferenced by a rejected call
    fwd = L.nb_linear_forward_ex
    assert fwd(None, None, P, P, None, 8, 8, 8, 0, None) == binding.NB_ERR_INVALID_ARG
    assert b"NULL" in L.nb_last_error()
    assert fwd(P, None, P, P, None, 8, 8, 8, 7, None) == binding.NB_ERR_INVALID_ARG
    assert fwd(P, None, P, P, None, -1, 8, 8, 0, None) == binding.NB_ERR_INVALID_ARG
    assert fwd(P, None, P, P, None, 8, 12, 8, 0, None) == binding.NB_ERR_UNSUPPORTED
    assert fwd(P, None, P, P, None, 8, 8, 20, 0, None) == binding.NB_ERR_UNSUPPORTED
    assert fwd(P + 2, None, P, P, None, 8, 8, 8, 0, None) == binding.NB_ERR_INVALID_ARG
    assert fwd(P, None, P, P, None, 8, 8, 24, binding.ACT_SWIGLU, None) == binding.NB_ERR_UNSUPPORTED
    assert fwd(P, None, P, P, None, 1 << 31, 8, 8, 0, None) == binding.NB_ERR_UNSUPPORTED
    bwd = L.nb_linear_backward_ex
    assert bwd(P, P, P, None, P, P, None, None, 8, 8, 8, 0, 0, 0, None) == binding.NB_ERR_INVALID_ARG
    assert bwd(P, P, P, P, P, P, None, None, 8, 8, 8, 1, 0, 0, None) == binding.NB_ERR_INVALID_ARG
    assert bwd(P, P, P, P, None, P, None, None, 8, 8, 8, 0, 0, 0, None) == binding.NB_ERR_INVALID_ARG
    assert bwd(P, P, P, P, P, None, None, None, 8, 8, 8, 0, 0, 0, None) == binding.NB_ERR_INVALID_ARG
    assert bwd(None, P, P, P, P, P, None, P, 8, 8, 8, 0, 0, 0, None) == binding.NB_ERR_INVALID_ARG
    assert bwd(P, P, P, P, P, P, None, None, 8, 8, 8, 0, 1, 1, None) == binding.NB_ERR_UNSUPPORTED
    assert bwd(P, P, P, P, P, P, None, None, 8, 8, 8, 0, 0, 5, None) == binding.NB_ERR_INVALID_ARG
    assert L.nb_reduce_dbias(None, P, 8, 8, 0) == binding.NB_ERR_INVALID_ARG
    assert L.nb_reduce_dbias(P, P, 8, 12, 0) == binding.NB_ERR_UNSUPPORTED
    assert L.nb_debug_wait_timeout(0) == binding.NB_ERR_INVALID_ARG
    assert L.nb_workspace_reserve(-5) == binding.NB_ERR_INVALID_ARG


def test_forward_with_zero_rows_is_a_no_op_everywhere(L):
    P = 0x10000
    assert L.nb_linear_forward_ex(P, None, P, P, None, 0, 8, 8, 0, None) == binding.NB_OK


def test_binding_has_no_cpu_path(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="missing"):
        binding.lib()


def test_wgrad_split_plan_covers_every_k_block_once(L):
    """Host logic: whatever split-K factor is chosen, the units partition (tile, k-block) space."""
    shapes_ = [(2304, 768, 16384), (768, 768, 16384), (3072, 768, 16384), (768, 3072, 16384),
               (50304, 768, 16384), (1024, 1024, 16384), (6144, 1024, 16384), (200, 72, 136),
               (3072, 768, 128), (8, 8, 1), (776, 328, 5000)]
    for M, N, K in shapes_:
        for slots, tile_m in ((148, 128), (74, 256)):
            tm, tn, splits, kps, kblocks = binding.nb_debug_split_plan(M, N, K, slots, tile_m)
            assert tm == -(-M // tile_m) and tn == -(-N // 256) and kblocks == -(-K // 64)
            assert 1 <= splits <= kblocks and kps >= 1
            covered = [0] * kblocks
            for s in range(splits):
                lo, hi = s * kps, min((s + 1) * kps, kblocks)
                assert lo < hi, "empty split"
                for kb in range(lo, hi):
                    covered[kb] += 1
            assert covered == [1] * kblocks
            # the chosen factor never leaves more than a wave's worth of imbalance on big problems
            if kblocks >= 64 and tm * tn <= slots:
                assert tm * tn * splits >= slots // 2


def test_layer_backward_plan_covers_every_unit_once(L):
    """Host logic of the one-launch layer backward: over all CTA pairs, every dinp tile appears once
    with its whole K range, and every (dweight tile, k-block) is covered exactly once, whatever
    the interleaving and the balancing cuts; loads are level across the pairs."""
    cases = [  # BT, C, OC
        (16384, 768, 2304), (16384, 768, 768), (16384, 768, 3072), (16384, 3072, 768),
        (16384, 768, 50304), (4096, 768, 3072), (4096, 3072, 768), (16384, 1024, 2048),
        (16384, 3072, 1024), (384, 768, 768), (136, 72, 200), (5000, 328, 776), (256, 8, 8),
    ]
    for BT, C, OC in cases:
        for pairs in (74, 66, 1):
            for gelu in (False, True):
                try:
                    hdr, recs = binding.nb_debug_layer_bwd_plan(BT, C, OC, pairs, gelu)
                except binding.NbError as e:
                    assert e.code == binding.NB_ERR_UNSUPPORTED and pairs == 1
                    continue
                dtm, dtn, dkb, wtm, wtn, wkb, kbc, rounds = hdr
                assert (dtm, dtn, dkb) == (-(-BT // 256), -(-C // 256), -(-OC // 64))
                assert (wtm, wtn, wkb) == (-(-OC // 256), -(-C // 256), -(-BT // 64))
                assert 1 <= kbc <= wkb and rounds <= 64
                d_seen = {}
                w_cov = {}
                load = [0] * pairs   # in the planner's cost units: k-blocks plus an allowance per unit
                for pr, is_w, m, n, kb0, kb1 in recs:
                    assert 0 <= pr < pairs and kb0 < kb1
                    load[pr] += kb1 - kb0 + (3 if is_w else (8 if gelu else 3))
                    if is_w:
                        assert 0 <= m < wtm and 0 <= n < wtn and kb1 <= wkb
                        cov = w_cov.setdefault((m, n), [0] * wkb)
                        for kb in range(kb0, kb1):
                            cov[kb] += 1
                    else:
                        assert 0 <= m < dtm and 0 <= n < dtn and (kb0, kb1) == (0, dkb)
                        d_seen[(m, n)] = d_seen.get((m, n), 0) + 1
                assert len(d_seen) == dtm * dtn and set(d_seen.values()) == {1}
                assert len(w_cov) == wtm * wtn
                assert all(c == [1] * wkb for c in w_cov.values())
                if pairs > 1 and BT >= 4096:
                    # level to within a few k-blocks (cuts are rounded to four, a cut unit pays
                    # its allowance twice)
                    assert max(load) - min(load) <= 16, (BT, C, OC, pairs, gelu, max(load), min(load))


def test_layer_backward_plan_on_drawn_shapes(L):
    """The same partition property on 200 drawn problems (seeded): row counts from just past one tile to
    70,000, widths from 8 to 6144, several pair counts. Either the planner declines (more rounds than its
    order mask holds) or every dinp tile appears once and every (dweight tile, k-block) exactly once."""
    import numpy as np
    rng = np.random.default_rng(20260928)
    declined = 0
    for case in range(200):
        BT = int(rng.integers(129, 70_000)) if case % 4 else int(rng.choice((129, 256, 257, 4096, 16384, 65536)))
        C = 8 * int(rng.integers(1, 769))
        OC = 8 * int(rng.integers(1, 769))
        pairs = int(rng.choice((74, 66, 33, 7)))
        gelu = bool(rng.integers(0, 2))
        try:
            hdr, recs = binding.nb_debug_layer_bwd_plan(BT, C, OC, pairs, gelu)
        except binding.NbError as e:
            assert e.code == binding.NB_ERR_UNSUPPORTED
            declined += 1
            continue
        dtm, dtn, dkb, wtm, wtn, wkb, kbc, rounds = hdr
        tag = (BT, C, OC, pairs, gelu)
        assert (dtm, dtn, dkb) == (-(-BT // 256), -(-C // 256), -(-OC // 64)), tag
        assert (wtm, wtn, wkb) == (-(-OC // 256), -(-C // 256), -(-BT // 64)), tag
        d_seen = np.zeros((dtm, dtn), dtype=np.int64)
        w_cov = np.zeros((wtm, wtn, wkb), dtype=np.int64)
        for pr, is_w, m, n, kb0, kb1 in recs:
            assert 0 <= pr < pairs and kb0 < kb1, tag
            if is_w:
                assert kb1 <= wkb, tag
                w_cov[m, n, kb0:kb1] += 1
            else:
                assert (kb0, kb1) == (0, dkb), tag
                d_seen[m, n] += 1
        assert (d_seen == 1).all(), tag
        assert (w_cov == 1).all(), tag
    assert declined < 100   # the drawn set mostly exercises the planner, not its refusal
