"""The C-ABI library loads, exports every symbol declared in include/lca.h, and rejects invalid
calls on the host before any launch (no GPU needed: nothing here reaches a kernel)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2604_12452_b200 import build
    build.build()
    from paper_2604_12452_b200 import binding
    return binding


def declared_functions():
    src = open(os.path.join(ROOT, "include", "lca.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(lca_[a-z_0-9]+)\s*\(", src)))


def test_header_declares_the_three_hot_path_calls():
    names = declared_functions()
    for n in ("lca_condense", "lca_prefill_attention", "lca_decode_attention", "lca_workspace_bytes"):
        assert n in names


def test_every_declared_symbol_is_exported(B):
    lib = C.CDLL(B._build.LIB)
    for name in declared_functions():
        assert hasattr(lib, name), name
    assert B.lca_version() >= 100
    assert B.lca_status_string(0) == "ok"
    assert "workspace" in B.lca_status_string(-4)


def test_partition_matches_section_4_2(B):
    p = B.make_params("mla", 1, 131072, 128, 1, 512, 64, 64, 4096, 0.07)
    assert B.lca_partition(p) == (1984, 4096)
    p = B.make_params("mla", 1, 1024, 4, 1, 512, 64, 64, 1024, 0.07)
    assert B.lca_partition(p) == (0, 1024)
    p = B.make_params("mla", 1, 1000, 4, 1, 512, 64, 64, 128, 0.07)
    assert B.lca_partition(p) == (13, 168)


def test_ragged_layout_is_the_partition_of_every_sequence(B):
    # host-only helper: prefix sums of L_b, m_b + k_b and m_b (Sec. 4.2 per sequence)
    p = B.make_params("mla", 4, 2000, 16, 1, 512, 64, 16, 64, 0.07)
    tok, cache, grp = B.lca_varlen_layout(p, [1, 50, 777, 2000])
    assert tok == [0, 1, 51, 828, 2828]
    ms = [0, 0, (777 - 64) // 16, (2000 - 64) // 16]
    ks = [1, 50, 777 - 16 * ms[2], 2000 - 16 * ms[3]]
    assert grp == [0, 0, 0, ms[2], ms[2] + ms[3]]
    assert cache == [0, 1, 51, 51 + ms[2] + ks[2], 51 + ms[2] + ks[2] + ms[3] + ks[3]]
    with pytest.raises(B.LcaError):
        B.lca_varlen_layout(p, [1, 0, 5, 7])               # lengths must be positive
    assert B.lca_workspace_bytes(p, B.LCA_WS_PREFILL_VARLEN) > 0 and B.lca_workspace_bytes(p, B.LCA_WS_CONDENSE_VARLEN) > 0


def test_invalid_calls_return_error_codes_without_launching(B):
    before = B.lca_launch_count()
    good = B.make_params("mla", 1, 1024, 4, 1, 512, 64, 64, 128, 0.07)
    assert B.lca_workspace_bytes(good, B.LCA_WS_CONDENSE) > 0
    # NULL tensors
    assert B.lca_condense(good, None, None, 64, None, None, None, None, None, None, None, None, 0) == -1
    assert B.lca_prefill_attention(good, None, None, None, None, None, None, None, None, None, 0) == -1
    assert B.lca_decode_attention(good, None, None, None, None, None, 16, 0, None, None, None, 0) == -1
    # bad parameters
    bad = B.make_params("mla", 1, 1024, 4, 2, 512, 64, 64, 128, 0.07)      # MLA has one KV stream
    assert B.lca_condense(bad, 16, 16, 64, None, 16, 16, 16, 16, 16, None, 16, 1 << 20) == -1
    bad = B.make_params("gqa", 1, 1024, 6, 4, 128, 128, 64, 128, 0.07)     # 6 % 4 != 0
    assert B.lca_prefill_attention(bad, None, 16, 16, 16, 16, 16, 16, None, None, 0) == -1
    bad = B.make_params("mla", 1, 1024, 4, 1, 512, 64, 0, 128, 0.07)       # g = 0
    assert B.lca_condense(bad, 16, 16, 64, None, 16, 16, 16, 16, 16, None, 16, 1 << 20) == -1
    bad = B.make_params("mla", 1, 1024, 4, 1, 500, 64, 64, 128, 0.07)      # rows not 16-byte multiples
    assert B.lca_condense(bad, 16, 16, 64, None, 16, 16, 16, 16, 16, None, 16, 1 << 20) == -2
    # misaligned pointer, too small a workspace, summary stride shorter than the tail
    assert B.lca_condense(good, 16, 16, 64, None, 24, 16, 16, 16, 16, None, 16, 1 << 20) == -3
    assert B.lca_condense(good, 16, 16, 64, None, 16, 16, 16, 16, 16, None, 16, 8) == -4
    assert B.lca_condense(good, 16, 16, 8, None, 16, 16, 16, 16, 16, None, 16, 1 << 20) == -1
    # shapes no attention kernel is built for
    odd = B.make_params("mla", 1, 1024, 4, 1, 256, 32, 64, 128, 0.07)
    assert B.lca_prefill_attention(odd, 16, 16, 16, 16, 16, 16, 16, None, None, 0) == -2
    assert B.lca_launch_count() == before


def test_ring_calls_reject_invalid_arguments_without_launching(B):
    # the ring layout needs whole groups to leave the ring (window % group_size == 0) and a buffer that holds the ring
    before = B.lca_launch_count()
    good = B.make_params("mla", 2, 0, 16, 1, 512, 64, 16, 48, 0.07)
    R = 48 + 16
    assert B.lca_ring_from_packed(good, None, 16, 16, 16, 80, 16, 16, R + 4, 16) == -1            # NULL packed cache
    assert B.lca_ring_from_packed(good, 16, 16, 16, 16, 80, 16, 16, R - 1, 16) == -1              # buffer smaller than the ring
    assert B.lca_ring_from_packed(good, 16, 16, 16, 16, 80, 24, 16, R + 4, 16) == -3              # misaligned ring buffer
    assert B.lca_decode_attention_ring(good, 16, 16, 16, 16, None, 16, R + 4, 16, None, None, 0) == -1   # NULL n_rep
    assert B.lca_decode_update_ring(good, 16, 16, 16, None, 16, 16, R + 4, 16, None, 16, 16, 1 << 20) == -1   # NULL n_tok
    assert B.lca_decode_update_ring(good, 16, 16, 16, None, 16, 16, R + 4, 16, 16, 16, 16, 8) == -4      # workspace too small
    assert B.lca_decode_step_update_ring(good, 16, 16, None, 16, 16, 16, R + 4, 16, 16, 16, 16, 1 << 20) == -1   # NULL running sum
    ragged_window = B.make_params("mla", 2, 0, 16, 1, 512, 64, 16, 40, 0.07)                      # 40 % 16 != 0
    assert B.lca_decode_attention_ring(ragged_window, 16, 16, 16, 16, 16, 16, 80, 16, None, None, 0) == -1
    assert B.lca_decode_update_ring(ragged_window, 16, 16, 16, None, 16, 16, 80, 16, 16, 16, 16, 1 << 20) == -1
    few = B.make_params("mla", 2, 0, 16, 1, 512, 64, 16, 48, 0.07, )
    few.n_summary_q = 4                                                                            # the running sum spans update to update
    assert B.lca_decode_step_update_ring(few, 16, 16, 16, 16, 16, 16, R + 4, 16, 16, 16, 16, 1 << 20) == -1
    assert B.lca_launch_count() == before
