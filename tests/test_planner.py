"""Host-side checks of the projection planner (no GPU): whatever shape it is given, the plan must respect
the limits the kernel relies on - tensor memory, shared memory, ring depth, cluster size, tile widths."""
import itertools

import pytest

from paper_2609_12075_b200 import adit

SHAPES = [(n_tok, n_feat, k, dual)
          for n_tok in (1, 16, 17, 34, 51, 100, 255, 256, 257, 408, 800, 816, 1632, 3264, 4096)
          for (n_feat, k, dual) in ((2560, 1024, False), (1024, 2048, False), (4096, 1024, True), (1024, 4096, False),
                                    (4608, 1536, False), (1536, 1536, False), (6144, 1536, True), (1536, 6144, False),
                                    (384, 256, False), (256, 256, False), (1024, 256, True), (256, 1024, False),
                                    (128, 64, False), (100, 64, False))]


@pytest.mark.parametrize("sm_count", [148, 132, 16])
def test_plan_limits(sm_count):
    for n_tok, n_feat, k, dual in SHAPES:
        p = adit.debug_plan(n_tok, n_feat, k, dual, sm_count)
        nv = 2 if dual else 1
        what = (n_tok, n_feat, k, dual, sm_count, p)
        assert p["tile_tok"] % 16 == 0 and 16 <= p["tile_tok"] <= 256, what
        assert p["n_ttiles"] * p["tile_tok"] >= n_tok, what                      # every token is covered
        assert p["n_ttiles"] * p["tile_tok"] - n_tok < 320, what                 # the buffers' padding rows suffice
        assert p["n_ftiles"] * 128 >= n_feat and p["kb_total"] == k // 64, what
        assert p["splits"] in (1, 2, 4, 8) and p["splits"] <= p["kb_total"], what
        if p["splits"] > 1:
            assert p["tile_tok"] % (8 * p["splits"]) == 0, what                 # every block finalises whole groups of 8 tokens
            assert p["n_ftiles"] * p["n_ttiles"] * p["splits"] <= sm_count, what  # clusters of a k-split run as one wave
        assert p["issuers"] in (1, 2) and p["acc_bufs"] in (1, 2), what
        assert p["acc_bufs"] * nv * p["issuers"] * p["tile_tok"] <= p["tmem_cols"] <= 512, what
        assert p["tmem_cols"] >= 32 and p["tmem_cols"] & (p["tmem_cols"] - 1) == 0, what
        if p["issuers"] == 2:
            assert p["stages"] % 2 == 0, what                                   # a stage must always belong to the same issuer
            assert p["kb_total"] // p["splits"] >= 2, what                      # both issuers have a k-block in every tile
        if p["acc_bufs"] == 1:
            assert p["n_ftiles"] * p["n_ttiles"] * p["splits"] <= sm_count, what
        assert 2 <= p["stages"] <= 12, what
        stage = nv * 128 * 64 * 2 + p["tile_tok"] * 64 * 2
        assert p["ring_bytes"] == p["stages"] * stage, what
        xbuf = 2 * p["tile_tok"] * 128 * 4 * nv if p["splits"] > 1 else 0
        assert p["smem_bytes"] == p["ring_bytes"] + xbuf + 1024 <= 217 * 1024, what


def test_plan_is_deterministic_and_rejects_bad_arguments():
    a = adit.debug_plan(816, 2560, 1024)
    assert a == adit.debug_plan(816, 2560, 1024)
    for bad in ((0, 128, 64), (16, 0, 64), (16, 128, 0), (16, 128, 100)):
        with pytest.raises(adit.AditError):
            adit.debug_plan(*bad)


@pytest.mark.parametrize("sm_count", [148, 132, 16, 2])
def test_projection_plan_uses_the_two_sm_kernel_only_where_it_may(sm_count):
    for n_tok, n_feat, k, dual in SHAPES + [(n, 4096, 1024, True) for n in (1023, 1024, 1025, 2000, 8192)]:
        one = adit.debug_plan(n_tok, n_feat, k, dual, sm_count)
        off = adit.debug_plan_projection(n_tok, n_feat, k, dual, sm_count, allow_pair=False)
        assert off.pop("pair") == 0 and off == one                              # the flag that forbids it gives the one-SM plan
        p = adit.debug_plan_projection(n_tok, n_feat, k, dual, sm_count)
        what = (n_tok, n_feat, k, dual, sm_count, p)
        if not (dual and n_tok >= 1024 and k >= 128):
            assert p.pop("pair") == 0 and p == one, what
            continue
        assert p["pair"] == 1 and p["splits"] == 1 and p["issuers"] == 1, what
        assert p["tile_tok"] % 16 == 0 and 32 <= p["tile_tok"] <= 256, what     # each block brings in half: whole 8-row groups
        assert p["n_ttiles"] * p["tile_tok"] >= n_tok, what
        assert p["n_ttiles"] * p["tile_tok"] - n_tok < 320, what
        assert p["acc_bufs"] in (1, 2) and p["acc_bufs"] * 2 * p["tile_tok"] <= p["tmem_cols"] <= 512, what
        stage = 2 * 128 * 64 * 2 + (p["tile_tok"] // 2) * 64 * 2                # this block's weight rows + its half of the tokens
        assert 2 <= p["stages"] <= 12 and p["ring_bytes"] == p["stages"] * stage, what
        assert p["smem_bytes"] == p["ring_bytes"] + 1024 <= 217 * 1024, what
