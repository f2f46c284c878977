"""lca_condense_static_scratch: the condensation for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a serving process whose
GPU memory was carved up once at start-up, in a latency-critical loop that must not take the
allocator's lock or trigger the implicit device synchronisation an allocation can cause.  For
them the library carries its own 1 MiB scratch array; this test checks, through the C ABI, that
the entry point built on it writes exactly what lca_condense writes, twice in a row (the second
call finds the first call's leftovers in the array), and that a problem too large for the array
is refused with its own status code before anything is launched.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.  It also passes on its own in a fresh process.
"""
import pytest
import torch

from paper_2604_12452_b200 import inputs as I

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def B():
    from paper_2604_12452_b200 import build
    build.build()
    from paper_2604_12452_b200 import binding
    return binding


def _outputs(B, p, dev):
    m, k = B.lca_partition(p)
    return dict(cache_sem=torch.full((p.batch, m + k, p.n_kv_heads, p.d_sem), 7.0, dtype=torch.bfloat16, device=dev),
                cache_pos=torch.full((p.batch, m + k, p.n_kv_heads, p.d_pos), 7.0, dtype=torch.bfloat16, device=dev),
                anchor_idx=torch.full((p.batch, max(m, 1), p.n_kv_heads), -1, dtype=torch.int32, device=dev)), m


def _both_ways(B, cfg, want_scores, first_call_on_device=False):
    inp = {k: v.to(DEV) for k, v in I.make_mla_inputs(cfg, "cpu").items()}
    p = B.params_from_config(cfg, batch=1)
    L, g = cfg.seq_len, cfg.group_size
    n = min(L, g)
    tail_sem, tail_pos = inp["q_sem"][L - n:].contiguous(), inp["q_pos"][L - n:].contiguous()
    ref, m = _outputs(B, p, DEV)
    got, _ = _outputs(B, p, DEV)
    sc_ref = torch.zeros((1, 1, max(m, 1) * g), dtype=torch.float64, device=DEV) if want_scores else None
    sc_got = torch.zeros_like(sc_ref) if want_scores else None
    ws = B.workspace(p, B.LCA_WS_CONDENSE, DEV)
    assert B.lca_condense(p, tail_sem, tail_pos, n, None, inp["ckv"], inp["kr"], ref["cache_sem"], ref["cache_pos"],
                          ref["anchor_idx"], sc_ref, ws) == 0
    before = B.lca_launch_count()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]          # the driver's count of free device bytes
    assert B.lca_condense_static_scratch(p, tail_sem, tail_pos, n, None, inp["ckv"], inp["kr"], got["cache_sem"],
                                         got["cache_pos"], got["anchor_idx"], sc_got) == 0
    assert B.lca_launch_count() > before
    torch.cuda.synchronize()
    if not first_call_on_device:
        # nothing was allocated or freed behind the caller's back (the very first call may page in the
        # library's kernels, which the driver accounts to the context, so it is left out)
        assert torch.cuda.mem_get_info()[0] == free_before
    # same kernels, same arithmetic, only the scratch lives elsewhere: the tolerance of the other
    # condense tests (bit-exact anchors and copies, c_rep within one bf16 ulp) tightens to equality
    for key in ref:
        assert torch.equal(ref[key], got[key]), key
    if want_scores:
        assert torch.equal(sc_ref, sc_got)


def test_static_scratch_condense_matches_lca_condense_twice_in_a_row(B):
    big = I.scaled(I.CONFIGS["mla_1k"], seq_len=2048, n_q_heads=128, group_size=64, window=256)
    small = I.scaled(I.CONFIGS["mla_1k"], seq_len=777, n_q_heads=16, group_size=16, window=100)
    assert 0 < B.lca_workspace_bytes(B.params_from_config(big, batch=1), B.LCA_WS_CONDENSE) <= B.LCA_STATIC_SCRATCH_BYTES
    _both_ways(B, big, want_scores=True, first_call_on_device=True)       # first call on this device: looks the array up
    _both_ways(B, small, want_scores=False)    # second call: the array still holds the first call's data


def test_static_scratch_condense_refuses_what_does_not_fit(B):
    p = B.make_params("mla", 64, 65536, 128, 1, 512, 64, 64, 4096, 0.07)
    assert B.lca_workspace_bytes(p, B.LCA_WS_CONDENSE) > B.LCA_STATIC_SCRATCH_BYTES
    before = B.lca_launch_count()
    st = B.lca_condense_static_scratch(p, 16, 16, 64, None, 16, 16, 16, 16, 16, None)
    assert st == B.LCA_ERR_STATIC_SCRATCH_EXCEEDED
    assert "LCA_STATIC_SCRATCH_BYTES" in B.lca_status_string(st)
    assert B.lca_launch_count() == before
