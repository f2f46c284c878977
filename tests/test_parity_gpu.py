"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the same seeded bits.

Small cases are compared element by element on every row; they span several KV tiles, a ragged
tail and the degenerate partitions (no group, window 0, sequence shorter than a group, ...).
"""
import math

import numpy as np
import pytest
import torch

from oracle import lca_oracle as O
from paper_2604_12452_b200 import inputs as I
from tests import helpers as Hh

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def B():
    from paper_2604_12452_b200 import build
    build.build()
    from paper_2604_12452_b200 import binding
    return binding


def to_dev(inp):
    return {k: v.to(DEV) for k, v in inp.items()}


def to_cpu(inp):
    return {k: v.cpu() for k, v in inp.items()}


def run_mla(B, cfg, inp_dev, n_summary=0, bias=0.0, impl=0, want_scores=True):
    p = B.params_from_config(cfg, batch=1, n_summary_q=n_summary, rep_logit_bias=bias)
    L = cfg.seq_len
    n = min(L, n_summary if n_summary > 0 else cfg.group_size)
    qs, qp = inp_dev["q_sem"], inp_dev["q_pos"]
    cond = B.condense(p, qs[L - n:], qp[L - n:], inp_dev["ckv"], inp_dev["kr"], want_scores=want_scores)
    prev = B.lca_set_attention_impl(impl)
    try:
        out, lse = B.prefill_attention(p, qs, qp, inp_dev["ckv"], inp_dev["kr"], cond["cache_sem"],
                                       cond["cache_pos"], want_lse=True)
    finally:
        B.lca_set_attention_impl(prev)
    torch.cuda.synchronize()
    return p, cond, out, lse


def one_seq(cond):
    r = dict(cond)
    for key in ("cache_sem", "cache_pos", "anchor_idx"):
        r[key] = cond[key][0]
    return r


MLA_SMALL = [
    # (L, H, g, w, n_summary)  -- d_c = 512, d_R = 64 throughout
    (1024, 4, 64, 128, 0),      # config 1 as given
    (1024, 4, 64, 1024, 0),     # paper-default window: no group, plain MLA
    (1000, 4, 64, 128, 0),      # ragged: (L - w) mod g = 40 residual tokens
    (777, 16, 16, 100, 32),     # paper-default group size, odd sizes, 32 summary queries
    (300, 128, 8, 64, 8),       # many heads (one token per 128-row tile)
    (130, 4, 64, 0, 0),         # window 0
    (50, 4, 64, 16, 0),         # shorter than one group
    (1, 4, 4, 0, 0),            # a single token
]


@pytest.mark.parametrize("L,H,g,w,ns", MLA_SMALL)
def test_mla_small_cases_match_oracle_on_every_row(B, L, H, g, w, ns):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=L, n_q_heads=H, group_size=g, window=w, n_needles=min(8, L))
    inp = I.make_mla_inputs(cfg, "cpu")
    p, cond, out, lse = run_mla(B, cfg, to_dev(inp), n_summary=ns)
    ref = Hh.oracle_mla(inp, g, w, cfg.softmax_scale, rows=np.arange(L), n_summary=ns)
    Hh.check_condense(one_seq(cond), ref["cond"])
    if ref["cond"]["m"]:
        sc = cond["scores"][0, 0].cpu().numpy()
        np.testing.assert_allclose(sc, ref["cond"]["scores"], rtol=0, atol=1e-12)
    Hh.check_outputs(out[0], ref, f"mla L={L} H={H} g={g} w={w}")
    np.testing.assert_allclose(lse[0].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4)


def test_mla_stress_peaky_queries_and_exact_ties(B):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=1024, n_q_heads=4)
    inp = I.stress_duplicate_tokens(I.stress_peaky_queries(I.make_mla_inputs(cfg, "cpu"), cfg), cfg)
    p, cond, out, _ = run_mla(B, cfg, to_dev(inp))
    ref = Hh.oracle_mla(inp, cfg.group_size, cfg.window, cfg.softmax_scale, rows=np.arange(cfg.seq_len))
    # the softmax is far from uniform here, and duplicated tokens tie exactly: lowest index wins
    alpha = ref["cond"]["alpha"].reshape(-1, cfg.group_size)
    assert alpha.max() > 0.5
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0], ref, "mla stress")


def test_mla_zero_queries_give_mean_pooling(B):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=512, n_q_heads=4)
    inp = I.make_mla_inputs(cfg, "cpu")
    inp["q_sem"] = torch.zeros_like(inp["q_sem"])
    inp["q_pos"] = torch.zeros_like(inp["q_pos"])
    p, cond, out, _ = run_mla(B, cfg, to_dev(inp))
    ref = Hh.oracle_mla(inp, cfg.group_size, cfg.window, cfg.softmax_scale, rows=np.arange(cfg.seq_len))
    m = ref["cond"]["m"]
    assert np.array_equal(ref["cond"]["anchor"], np.arange(m) * cfg.group_size)
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0], ref, "mla q=0")


def test_mla_rep_logit_bias_and_supplied_summary_query(B):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=640, n_q_heads=4, group_size=16, window=64)
    inp = I.make_mla_inputs(cfg, "cpu")
    d = to_dev(inp)
    bias = math.log(cfg.group_size)
    qbar32 = torch.randn(1, 1, 576, generator=torch.Generator().manual_seed(5)).float()
    p = B.params_from_config(cfg, batch=1, rep_logit_bias=bias)
    cond = B.condense(p, None, None, d["ckv"], d["kr"], qbar=qbar32.to(DEV), want_scores=True)
    out, _ = B.prefill_attention(p, d["q_sem"], d["q_pos"], d["ckv"], d["kr"], cond["cache_sem"], cond["cache_pos"])
    ref = Hh.oracle_mla(inp, cfg.group_size, cfg.window, cfg.softmax_scale, rows=np.arange(cfg.seq_len),
                        rep_logit_bias=bias, qbar=qbar32[0, 0].double().numpy())
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0], ref, "mla bias=ln g")


def test_mla_batched_sequences_are_independent(B):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=384, n_q_heads=4, group_size=32, window=64, batch=3)
    seqs = [I.make_mla_inputs(cfg, "cpu", batch_index=b) for b in range(3)]
    stack = {k: torch.stack([s[k] for s in seqs]).to(DEV) for k in seqs[0]}
    p = B.params_from_config(cfg, batch=3)
    g = cfg.group_size
    # summary tail taken straight out of the full [B, L, H, d] query tensors (stride L)
    L = cfg.seq_len
    qs_tail = stack["q_sem"][:, L - g:].contiguous()
    qp_tail = stack["q_pos"][:, L - g:].contiguous()
    cond = B.condense(p, qs_tail, qp_tail, stack["ckv"], stack["kr"])
    out, _ = B.prefill_attention(p, stack["q_sem"], stack["q_pos"], stack["ckv"], stack["kr"],
                                 cond["cache_sem"], cond["cache_pos"])
    # the same through pointers into the full tensors: tail of sequence b starts L rows after b-1's
    p2 = B.params_from_config(cfg, batch=3)
    first_tail_sem = stack["q_sem"].data_ptr() + (L - g) * cfg.n_q_heads * cfg.d_sem * 2
    first_tail_pos = stack["q_pos"].data_ptr() + (L - g) * cfg.n_q_heads * cfg.d_pos * 2
    cond2 = B.condense(p2, first_tail_sem, first_tail_pos, stack["ckv"], stack["kr"], q_tail_batch_stride=L)
    assert torch.equal(cond["cache_sem"], cond2["cache_sem"]) and torch.equal(cond["anchor_idx"], cond2["anchor_idx"])
    for b in range(3):
        ref = Hh.oracle_mla(seqs[b], g, cfg.window, cfg.softmax_scale, rows=np.arange(L))
        r = dict(cond)
        for key in ("cache_sem", "cache_pos", "anchor_idx"):
            r[key] = cond[key][b]
        Hh.check_condense(r, ref["cond"])
        Hh.check_outputs(out[b], ref, f"batch {b}")


@pytest.mark.parametrize("H", [1, 2, 8, 32, 64, 256])
def test_mla_head_counts_of_the_pair_kernel(B, H):
    # Every way a 128-row tile of the CTA-pair kernel splits into tokens x heads: H < 128 puts 128 / H tokens in
    # a tile (H = 1: 64 tokens per CTA), H = 256 two head blocks per token.  Every row, tensor-core path forced.
    L, g, w = 333, 16, 50
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=L, n_q_heads=H, group_size=g, window=w, n_needles=4)
    inp = I.make_mla_inputs(cfg, "cpu")
    p, cond, out, lse = run_mla(B, cfg, to_dev(inp), impl=2, want_scores=False)
    ref = Hh.oracle_mla(inp, g, w, cfg.softmax_scale, rows=np.arange(L))
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0], ref, f"mla H={H}")
    np.testing.assert_allclose(lse[0].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4)
    assert B.lca_last_device_status() == 0


GQA_SMALL = [(1024, 32, 8, 64, 128), (515, 8, 2, 16, 40), (96, 4, 4, 64, 64), (260, 32, 8, 64, 0)]


@pytest.mark.parametrize("L,Hq,Hkv,g,w", GQA_SMALL)
def test_gqa_small_cases_match_oracle_on_every_row(B, L, Hq, Hkv, g, w):
    cfg = I.scaled(I.CONFIGS["gqa_64k"], seq_len=L, n_q_heads=Hq, n_kv_heads=Hkv, group_size=g, window=w,
                   n_needles=4)
    inp = I.make_gqa_inputs(cfg, "cpu")
    d = to_dev(inp)
    p = B.params_from_config(cfg, batch=1)
    n = min(L, g)
    cond = B.condense(p, None, d["q"][L - n:], d["v"], d["k"], want_scores=True)
    out, lse = B.prefill_attention(p, None, d["q"], d["v"], d["k"], cond["cache_sem"], cond["cache_pos"],
                                   want_lse=True)
    assert B.lca_last_device_status() == 0
    ref = Hh.oracle_gqa(inp, g, w, cfg.softmax_scale, rows=np.arange(L))
    Hh.check_condense(one_seq(cond), ref["cond"], kind="gqa")
    Hh.check_outputs(out[0], ref, f"gqa L={L}")
    np.testing.assert_allclose(lse[0].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4)


def test_output_pointer_aligned_to_16_bytes_only(B):
    # The ABI promises 16-byte alignment, the tensor-core kernels store 32 bytes at a time where they can:
    # an output buffer that starts 16 bytes into an allocation must give the same bits as an aligned one.
    def shifted(shape):
        n = int(np.prod(shape))
        raw = torch.zeros(n + 8, dtype=torch.bfloat16, device=DEV)
        view = raw[8:].view(shape)
        assert view.data_ptr() % 32 == 16
        return view

    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=300, n_q_heads=16, group_size=16, window=64)
    d = to_dev(I.make_mla_inputs(cfg, "cpu"))
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, d["q_sem"][300 - 16:], d["q_pos"][300 - 16:], d["ckv"], d["kr"])
    args = (p, d["q_sem"], d["q_pos"], d["ckv"], d["kr"], cond["cache_sem"], cond["cache_pos"])
    ref, _ = B.prefill_attention(*args)
    out, _ = B.prefill_attention(*args, out=shifted((1, 300, 16, 512)))
    assert torch.equal(Hh.bits_t(out), Hh.bits_t(ref))

    cfg = I.scaled(I.CONFIGS["gqa_64k"], seq_len=260, n_q_heads=8, n_kv_heads=2, group_size=16, window=40)
    d = to_dev(I.make_gqa_inputs(cfg, "cpu"))
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, None, d["q"][260 - 16:], d["v"], d["k"])
    args = (p, None, d["q"], d["v"], d["k"], cond["cache_sem"], cond["cache_pos"])
    ref, _ = B.prefill_attention(*args)
    out, _ = B.prefill_attention(*args, out=shifted((1, 260, 8, 128)))
    assert torch.equal(Hh.bits_t(out), Hh.bits_t(ref))
    assert B.lca_last_device_status() == 0


def test_mla_decode_matches_oracle_and_prefill_row(B):
    # contexts of different lengths share one cache buffer (capacity = longest + 1 appended row)
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=3, seq_len=1500, n_q_heads=128, group_size=64, window=256)
    g, w, H = cfg.group_size, cfg.window, cfg.n_q_heads
    p = B.params_from_config(cfg, batch=3)
    m, k = B.lca_partition(p)
    cap = m + k + 1
    cache_sem = torch.zeros((3, cap, 1, 512), dtype=torch.bfloat16, device=DEV)
    cache_pos = torch.zeros((3, cap, 1, 64), dtype=torch.bfloat16, device=DEV)
    rows = torch.tensor([m + k + 1, m + k + 1, m + k - 5], dtype=torch.int32, device=DEV)
    q_new_sem = torch.randn((3, H, 512), generator=torch.Generator().manual_seed(1)).bfloat16()
    q_new_pos = torch.randn((3, H, 64), generator=torch.Generator().manual_seed(2)).bfloat16()
    refs = []
    p1 = B.params_from_config(cfg, batch=1)
    for b in range(3):
        inp = I.make_mla_inputs(cfg, "cpu", batch_index=b, q_positions=slice(cfg.seq_len - g, cfg.seq_len))
        d = to_dev(inp)
        c = B.condense(p1, d["q_sem"], d["q_pos"], d["ckv"], d["kr"])
        ref = Hh.oracle_mla(inp, g, w, cfg.softmax_scale)
        Hh.check_condense(one_seq(c), ref["cond"])
        cache_sem[b, :m + k] = c["cache_sem"][0]
        cache_pos[b, :m + k] = c["cache_pos"][0]
        new_sem = torch.randn((1, 512), generator=torch.Generator().manual_seed(10 + b)).bfloat16()
        new_pos = torch.randn((1, 64), generator=torch.Generator().manual_seed(20 + b)).bfloat16()
        cache_sem[b, m + k, 0] = new_sem[0].to(DEV)
        cache_pos[b, m + k, 0] = new_pos[0].to(DEV)
        nrows = int(rows[b])
        cs = O.bits_to_f64(Hh.bits(cache_sem[b, :nrows, 0]))
        cp = O.bits_to_f64(Hh.bits(cache_pos[b, :nrows, 0]))
        refs.append(O.mla_decode(O.torch_bf16_to_f64(q_new_sem[b]), O.torch_bf16_to_f64(q_new_pos[b]), cs, cp,
                                 m, Hh.f32(cfg.softmax_scale)))
    out, lse = B.decode_attention(p, q_new_sem.to(DEV), q_new_pos.to(DEV), cache_sem, cache_pos, rows, m,
                                  want_lse=True)
    for b in range(3):
        Hh.check_outputs(out[b], refs[b][0], f"decode seq {b}")
        np.testing.assert_allclose(lse[b].cpu().numpy(), refs[b][1], atol=2e-3, rtol=1e-4)


def test_mla_many_query_tiles_per_cta_pair(B):
    # 128 heads: one token per 128-row tile, so 2000 work items for the ~74 resident CTA pairs of the persistent
    # kernel -- about 27 items per pair, of 1 to 8 key tiles each: item boundaries, the per-item barriers
    # wrapping many times, tile counts of both parities.  Sampled rows, every head.
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=2000, n_q_heads=128, group_size=16, window=300, n_needles=8)
    inp = I.make_mla_inputs(cfg, "cpu")
    p, cond, out, lse = run_mla(B, cfg, to_dev(inp), want_scores=False)
    L = cfg.seq_len
    rows = np.unique(np.concatenate([np.arange(0, L, 13), np.arange(0, 40), np.arange(L - 160, L)]))
    ref = Hh.oracle_mla(inp, cfg.group_size, cfg.window, cfg.softmax_scale, rows=rows)
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0][torch.from_numpy(rows).to(DEV)], ref, "mla many items per pair")
    np.testing.assert_allclose(lse[0].cpu().numpy()[rows], ref["lse"], atol=2e-3, rtol=1e-4)
    assert B.lca_last_device_status() == 0


def test_mla_decode_more_sequences_than_cta_pairs_with_empty_caches(B):
    # 100 sequences x 128 heads = 100 work items: some CTA pairs take two.  Row counts span several key-tile
    # counts; two sequences have an empty cache (no item work: zero output, lse = -inf).
    H, nb, cap = 128, 100, 700
    gen = torch.Generator().manual_seed(77)
    cache_sem = torch.randn((nb, cap, 1, 512), generator=gen).bfloat16()
    cache_pos = torch.randn((nb, cap, 1, 64), generator=gen).bfloat16()
    q_sem = torch.randn((nb, H, 512), generator=gen).bfloat16()
    q_pos = torch.randn((nb, H, 64), generator=gen).bfloat16()
    rows = torch.randint(1, cap + 1, (nb,), generator=gen, dtype=torch.int32)
    rows[5] = 0; rows[93] = 0; rows[7] = cap; rows[8] = 128; rows[9] = 129; rows[10] = 1
    n_rep = 40
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=nb, seq_len=4096, n_q_heads=H, group_size=64, window=256)
    p = B.params_from_config(cfg, batch=nb)
    out, lse = B.decode_attention(p, q_sem.to(DEV), q_pos.to(DEV), cache_sem.to(DEV), cache_pos.to(DEV),
                                  rows.to(DEV), n_rep, want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    for b in list(range(0, nb, 9)) + [5, 7, 8, 9, 10, 93]:
        n = int(rows[b])
        if n == 0:
            assert torch.count_nonzero(out[b]) == 0
            assert torch.isinf(lse[b]).all() and (lse[b] < 0).all()
            continue
        cs = O.bits_to_f64(Hh.bits(cache_sem[b, :n, 0]))
        cp = O.bits_to_f64(Hh.bits(cache_pos[b, :n, 0]))
        ro, rl = O.mla_decode(O.torch_bf16_to_f64(q_sem[b]), O.torch_bf16_to_f64(q_pos[b]), cs, cp,
                              min(n_rep, n), Hh.f32(cfg.softmax_scale))
        Hh.check_outputs(out[b], ro, f"decode seq {b} rows {n}")
        np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)


def test_dense_window_is_plain_causal_attention(B):
    # window >= L: the dense-MLA comparison run through the same entry point (Eq. 5), every row.
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=600, n_q_heads=16, window=600)
    inp = I.make_mla_inputs(cfg, "cpu")
    p, cond, out, _ = run_mla(B, cfg, to_dev(inp))
    assert cond["m"] == 0 and cond["k"] == 600
    ref = Hh.oracle_mla(inp, cfg.group_size, cfg.window, cfg.softmax_scale, rows=np.arange(600))
    Hh.check_outputs(out[0], ref, "dense")


def test_launches_are_counted(B):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=256, n_q_heads=4)
    inp = to_dev(I.make_mla_inputs(cfg, "cpu"))
    before = B.lca_launch_count()
    run_mla(B, cfg, inp)
    assert B.lca_launch_count() - before == 5     # 2 summary + condense + window copy + attention


def test_online_cache_update_matches_oracle_over_many_decode_steps(B):
    # three sequences in different phases of the buffer; 2 g + 5 generated tokens each, so every
    # sequence condenses two or three times; a fresh summary query (last g queries) at every step
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=3, seq_len=0, n_q_heads=16, group_size=16, window=40)
    g, w, H, Bsz = cfg.group_size, cfg.window, cfg.n_q_heads, 3
    cap = 8 + w + g + 4
    gen = torch.Generator().manual_seed(11)
    p = B.params_from_config(cfg, batch=Bsz)
    n_rep0 = [3, 5, 0]
    n_loc0 = [w + g - 1, w + 3, w]
    sem = torch.zeros((Bsz, cap, 1, 512), dtype=torch.bfloat16)
    pos = torch.zeros((Bsz, cap, 1, 64), dtype=torch.bfloat16)
    for b in range(Bsz):
        n = n_rep0[b] + n_loc0[b]
        sem[b, :n, 0] = torch.randn((n, 512), generator=gen).bfloat16()
        pos[b, :n, 0] = torch.randn((n, 64), generator=gen).bfloat16()
    d_sem, d_pos = sem.to(DEV), pos.to(DEV)
    d_nrep = torch.tensor(n_rep0, dtype=torch.int32, device=DEV)
    d_rows = torch.tensor([a + c for a, c in zip(n_rep0, n_loc0)], dtype=torch.int32, device=DEV)
    o_sem = [Hh.bits(sem[b, :, 0]) for b in range(Bsz)]
    o_pos = [Hh.bits(pos[b, :, 0]) for b in range(Bsz)]
    o_nrep, o_rows = list(n_rep0), [a + c for a, c in zip(n_rep0, n_loc0)]
    n_updates = 0
    for step in range(2 * g + 5):
        new_sem = torch.randn((Bsz, 512), generator=gen).bfloat16()
        new_pos = torch.randn((Bsz, 64), generator=gen).bfloat16()
        q_tail_sem = torch.randn((Bsz, g, H, 512), generator=gen).bfloat16()
        q_tail_pos = torch.randn((Bsz, g, H, 64), generator=gen).bfloat16()
        rows_now = d_rows.cpu().tolist()
        for b in range(Bsz):                       # the caller appends the new token's row
            d_sem[b, rows_now[b], 0] = new_sem[b].to(DEV)
            d_pos[b, rows_now[b], 0] = new_pos[b].to(DEV)
        d_rows += 1
        anchor = B.decode_update(p, q_tail_sem.to(DEV), q_tail_pos.to(DEV), d_sem, d_pos, d_nrep, d_rows)
        torch.cuda.synchronize()
        for b in range(Bsz):
            o_sem[b][o_rows[b]] = Hh.bits(new_sem[b])
            o_pos[b][o_rows[b]] = Hh.bits(new_pos[b])
            o_rows[b] += 1
            qbar = O.mla_summary_query(O.torch_bf16_to_f64(q_tail_sem[b]), O.torch_bf16_to_f64(q_tail_pos[b]))
            s2, p2, o_nrep[b], o_rows[b], ia = O.mla_decode_update(o_sem[b][:o_rows[b]], o_pos[b][:o_rows[b]], o_nrep[b],
                                                                 o_rows[b], qbar, g, w, Hh.f32(cfg.softmax_scale))
            o_sem[b] = np.concatenate([s2, np.zeros((cap - len(s2), 512), np.uint16)])
            o_pos[b] = np.concatenate([p2, np.zeros((cap - len(p2), 64), np.uint16)])
            n_updates += ia >= 0
            assert int(anchor[b, 0]) == ia
        assert d_nrep.cpu().tolist() == o_nrep and d_rows.cpu().tolist() == o_rows
        for b in range(Bsz):
            n, r = o_rows[b], o_nrep[b]
            got_sem, got_pos = Hh.bits(d_sem[b, :n, 0]), Hh.bits(d_pos[b, :n, 0])
            assert np.array_equal(got_pos, o_pos[b][:n])                       # anchors and tokens: bit copies
            assert np.array_equal(got_sem[r:], o_sem[b][r:n])                  # buffered tokens in order
            ulp = Hh.bf16_ulp_distance(got_sem[:r], o_sem[b][:r])
            assert (ulp <= 1).all()                                            # representatives: fp32 pooling
            o_sem[b][:r] = got_sem[:r]                                         # carry the device's rounding forward
    assert n_updates >= 6


REDUCERS = {"maxpool": 1, "meanpool": 2, "weighted": 3, "maxsel": 4}


@pytest.mark.parametrize("sem", list(REDUCERS))
@pytest.mark.parametrize("pos", list(REDUCERS))
def test_ablation_reducers_match_oracle(B, sem, pos):
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=400, n_q_heads=4, group_size=32, window=48)
    inp = I.stress_peaky_queries(I.make_mla_inputs(cfg, "cpu"), cfg)
    d = to_dev(inp)
    L, g = cfg.seq_len, cfg.group_size
    p = B.params_from_config(cfg, batch=1, sem_reducer=REDUCERS[sem], pos_reducer=REDUCERS[pos])
    cond = B.condense(p, d["q_sem"][L - g:], d["q_pos"][L - g:], d["ckv"], d["kr"])
    torch.cuda.synchronize()
    qbar = O.mla_summary_query(O.torch_bf16_to_f64(inp["q_sem"][L - g:]), O.torch_bf16_to_f64(inp["q_pos"][L - g:]))
    ref = O.mla_condense(qbar, O.torch_bf16_to_f64(inp["ckv"]), O.torch_bf16_to_f64(inp["kr"]), g, cfg.window,
                         Hh.f32(cfg.softmax_scale), sem, pos)
    m, k = ref["m"], ref["k"]
    got_sem, got_pos = Hh.bits(cond["cache_sem"][0, :, 0]), Hh.bits(cond["cache_pos"][0, :, 0])
    assert np.array_equal(cond["anchor_idx"][0, :, 0].cpu().numpy(), ref["anchor"])
    assert np.array_equal(got_sem[m:], ref["cache_sem_bits"][m:]) and np.array_equal(got_pos[m:], ref["cache_pos_bits"][m:])
    for got, want, mode in ((got_sem[:m], ref["cache_sem_bits"][:m], sem), (got_pos[:m], ref["cache_pos_bits"][:m], pos)):
        if mode in ("maxsel", "maxpool"):
            assert np.array_equal(got, want)                       # selections and maxima are exact
        else:
            ulp = Hh.bf16_ulp_distance(got, want)
            tiny = np.abs(O.bits_to_f64(got) - O.bits_to_f64(want)) <= 32 * 2.0 ** -24 * 20.0
            assert ((ulp <= 1) | tiny).all()                       # fp32 sums of g terms against fp64


def test_gqa_decode_matches_oracle(B):
    # GQA cache: K anchors / pooled V per KV head; sequences of different valid lengths share one buffer,
    # rows past the valid count are left as zeros (they take no part in the result)
    cfg = I.scaled(I.CONFIGS["gqa_64k"], batch=3, seq_len=900, n_q_heads=32, n_kv_heads=8, group_size=64, window=128)
    g, w, Hq, Hkv, d = cfg.group_size, cfg.window, cfg.n_q_heads, cfg.n_kv_heads, cfg.d_sem
    p1 = B.params_from_config(cfg, batch=1)
    m, k = B.lca_partition(p1)
    cap = m + k + 1
    cache_v = torch.zeros((3, cap, Hkv, d), dtype=torch.bfloat16, device=DEV)
    cache_k = torch.zeros((3, cap, Hkv, d), dtype=torch.bfloat16, device=DEV)
    valid = [m + k + 1, m + k - 37, m + 1]
    gen = torch.Generator().manual_seed(3)
    q_new = torch.randn((3, Hq, d), generator=gen).bfloat16()
    refs = []
    for b in range(3):
        inp = I.make_gqa_inputs(cfg, "cpu", batch_index=b)
        dv = to_dev(inp)
        c = B.condense(p1, None, dv["q"][cfg.seq_len - g:], dv["v"], dv["k"])
        ref = Hh.oracle_gqa(inp, g, w, cfg.softmax_scale)
        Hh.check_condense(one_seq(c), ref["cond"], kind="gqa")
        cache_v[b, :m + k] = c["cache_sem"][0]
        cache_k[b, :m + k] = c["cache_pos"][0]
        cache_v[b, m + k] = torch.randn((Hkv, d), generator=gen).bfloat16().to(DEV)
        cache_k[b, m + k] = torch.randn((Hkv, d), generator=gen).bfloat16().to(DEV)
        n = valid[b]
        refs.append(O.gqa_decode(O.torch_bf16_to_f64(q_new[b]), O.bits_to_f64(Hh.bits(cache_k[b, :n])),
                                 O.bits_to_f64(Hh.bits(cache_v[b, :n])), m, Hh.f32(cfg.softmax_scale), 0.25))
    p = B.params_from_config(cfg, batch=3, rep_logit_bias=0.25)
    rows = torch.tensor(valid, dtype=torch.int32, device=DEV)
    for impl in (0, 1):                                  # tensor-core kernel, then the scalar kernel
        prev = B.lca_set_attention_impl(impl)
        try:
            out, lse = B.decode_attention(p, None, q_new.to(DEV), cache_v, cache_k, rows, m, want_lse=True)
        finally:
            B.lca_set_attention_impl(prev)
        assert B.lca_last_device_status() == 0
        for b in range(3):
            Hh.check_outputs(out[b], refs[b][0], f"gqa decode seq {b} impl {impl}")
            np.testing.assert_allclose(lse[b].cpu().numpy(), refs[b][1], atol=2e-3, rtol=1e-4)


def test_decode_ignores_non_finite_rows_behind_the_valid_count(B):
    # Capacity rows at or behind cache_rows[b] may hold anything (here NaN and Inf bit patterns): they must not reach
    # the output (probability 0 times NaN is NaN).  Ragged counts, a count on a tile boundary, empty caches; the MLA
    # shape (CTA-pair kernel) and the GQA shape (one-CTA kernel).
    gen = torch.Generator().manual_seed(123)
    nb, cap, H = 6, 300, 128
    counts = [300, 299, 129, 128, 1, 0]
    cache_sem = torch.randn((nb, cap, 1, 512), generator=gen).bfloat16()
    cache_pos = torch.randn((nb, cap, 1, 64), generator=gen).bfloat16()
    q_sem = torch.randn((nb, H, 512), generator=gen).bfloat16()
    q_pos = torch.randn((nb, H, 64), generator=gen).bfloat16()
    poisoned_sem, poisoned_pos = cache_sem.clone(), cache_pos.clone()
    for b, n in enumerate(counts):
        poisoned_sem[b, n:] = float("nan")
        poisoned_pos[b, n:] = float("inf") if b % 2 else float("nan")
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=nb, seq_len=4096, n_q_heads=H)
    p = B.params_from_config(cfg, batch=nb)
    rows = torch.tensor(counts, dtype=torch.int32, device=DEV)
    out, lse = B.decode_attention(p, q_sem.to(DEV), q_pos.to(DEV), poisoned_sem.to(DEV), poisoned_pos.to(DEV), rows, 17,
                                  want_lse=True)
    assert B.lca_last_device_status() == 0
    assert torch.isfinite(out.float()).all()
    for b, n in enumerate(counts):
        if n == 0:
            assert torch.count_nonzero(out[b]) == 0
            continue
        ro, rl = O.mla_decode(O.torch_bf16_to_f64(q_sem[b]), O.torch_bf16_to_f64(q_pos[b]),
                              O.bits_to_f64(Hh.bits(cache_sem[b, :n, 0])), O.bits_to_f64(Hh.bits(cache_pos[b, :n, 0])),
                              min(17, n), Hh.f32(cfg.softmax_scale))
        Hh.check_outputs(out[b], ro, f"mla decode, {n} valid rows, NaN behind")
        np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)

    Hq, Hkv, d = 32, 8, 128
    ck = torch.randn((nb, cap, Hkv, d), generator=gen).bfloat16()
    cv = torch.randn((nb, cap, Hkv, d), generator=gen).bfloat16()
    q = torch.randn((nb, Hq, d), generator=gen).bfloat16()
    pk, pv = ck.clone(), cv.clone()
    for b, n in enumerate(counts):
        pk[b, n:] = float("nan")
        pv[b, n:] = float("nan")
    cfg = I.scaled(I.CONFIGS["gqa_64k"], batch=nb, seq_len=4096)
    p = B.params_from_config(cfg, batch=nb)
    out, _ = B.decode_attention(p, None, q.to(DEV), pv.to(DEV), pk.to(DEV), rows, 17)
    assert B.lca_last_device_status() == 0
    assert torch.isfinite(out.float()).all()
    for b, n in enumerate(counts):
        if n == 0:
            assert torch.count_nonzero(out[b]) == 0
            continue
        ro, _ = O.gqa_decode(O.torch_bf16_to_f64(q[b]), O.bits_to_f64(Hh.bits(ck[b, :n])), O.bits_to_f64(Hh.bits(cv[b, :n])),
                             min(17, n), Hh.f32(cfg.softmax_scale))
        Hh.check_outputs(out[b], ro, f"gqa decode, {n} valid rows, NaN behind")


def test_a_bounded_device_wait_that_expires_is_reported_and_harmless(B):
    # The library's own self-test kernel waits, with the routine every tensor-core kernel uses, on a barrier nobody
    # arrives on; after ~1e5 cycles it gives up, records the code and returns.  The status is reported once, and the
    # next ordinary call works.
    assert B.lca_last_device_status() == 0
    assert B.lca_selftest_bounded_wait(0) == -1 and B.lca_selftest_bounded_wait(10 ** 12) == -1      # limit out of range
    assert B.lca_selftest_bounded_wait(100_000) == 0
    assert B.lca_last_device_status() == B.LCA_ERR_DEVICE_TIMEOUT
    assert B.lca_last_device_status() == 0
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=300, n_q_heads=16, group_size=16, window=64)
    inp = I.make_mla_inputs(cfg, "cpu")
    p, cond, out, _ = run_mla(B, cfg, to_dev(inp), want_scores=False)
    assert B.lca_last_device_status() == 0
    ref = Hh.oracle_mla(inp, cfg.group_size, cfg.window, cfg.softmax_scale, rows=np.arange(cfg.seq_len))
    Hh.check_outputs(out[0], ref, "after an expired wait")


@pytest.mark.parametrize("T,H", [(300, 16), (128, 1), (1, 128), (1000, 3)])
def test_latent_to_value_matches_oracle(B, T, H):
    # out_v[t, h] = latent[t, h] W^UV[h]: several token tiles and a ragged last one, one head to many;
    # bf16 products, fp32 sums of 512 terms, one rounding of the result
    gen = torch.Generator().manual_seed(1000 + T)
    x = torch.randn((T, H, 512), generator=gen).bfloat16()
    W = (torch.randn((H, 512, 128), generator=gen) / 512 ** 0.5).bfloat16()
    W[H // 2] *= -2.0
    got = B.latent_to_value(x.to(DEV), W.to(DEV))
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    ref = O.latent_to_value(O.torch_bf16_to_f64(x), O.torch_bf16_to_f64(W))
    ulp = Hh.bf16_ulp_distance(Hh.bits(got), O.round_bf16_bits(ref))
    err = np.abs(got.float().cpu().numpy().astype(np.float64) - ref)
    # fp32 accumulation of 512 terms: absolute error <= 512 * 2^-24 * sum |x||w| (~1e-4 here), else one bf16 ulp
    assert ((ulp <= 1) | (err <= 2e-4)).all(), f"max ulp {ulp.max()}, max err {err.max()}"
    assert (ulp > 0).mean() < 0.02


def test_absorbed_attention_plus_value_projection_equals_unabsorbed_attention(B):
    # Alg. 1 builds k_rep = [c_rep W^UK, k^R_I] and v_rep = c_rep W^UV; the library works in the latent space with
    # q_latent = q_nope W^UK^T and applies W^UV to the attention result.  Against a numpy restatement of the
    # un-absorbed form on the same bf16 inputs (the representatives taken from the device cache).
    rng = np.random.default_rng(77)
    L, H, g, w, dn = 300, 16, 16, 40, 128
    scale = 1.0 / (dn + 64) ** 0.5
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=L, n_q_heads=H, group_size=g, window=w, n_needles=0, softmax_scale=scale)
    inp = I.make_mla_inputs(cfg, "cpu")
    WUK = torch.from_numpy(rng.standard_normal((H, 512, dn)) / 512 ** 0.5).bfloat16()
    WUV = torch.from_numpy(rng.standard_normal((H, 512, 128)) / 512 ** 0.5).bfloat16()
    q_nope = torch.from_numpy(rng.standard_normal((L, H, dn))).bfloat16()
    q_lat = torch.einsum("lhn,hcn->lhc", q_nope.float(), WUK.float()).bfloat16().contiguous()   # absorbed query, as the model would feed it
    inp["q_sem"] = q_lat
    d = to_dev(inp)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, d["q_sem"][L - g:], d["q_pos"][L - g:], d["ckv"], d["kr"])
    out, _ = B.prefill_attention(p, d["q_sem"], d["q_pos"], d["ckv"], d["kr"], cond["cache_sem"], cond["cache_pos"])
    out_v = B.latent_to_value(out, WUV.to(DEV))
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    m = cond["m"]
    C, KR = O.torch_bf16_to_f64(inp["ckv"]), O.torch_bf16_to_f64(inp["kr"])
    c_rep = O.bits_to_f64(Hh.bits(cond["cache_sem"][0, :m, 0]))
    kr_rep = O.bits_to_f64(Hh.bits(cond["cache_pos"][0, :m, 0]))
    wuk, wuv = O.torch_bf16_to_f64(WUK), O.torch_bf16_to_f64(WUV)
    qn, qr = O.torch_bf16_to_f64(q_nope), O.torch_bf16_to_f64(inp["q_pos"])
    rows = [0, 5, w + g - 2, w + g - 1, w + g, 150, L - 1]
    ref = np.zeros((len(rows), H, 128))
    for x, t in enumerate(rows):
        mt = 0 if t + 1 < w + g else (t + 1 - w) // g
        sem = np.concatenate([c_rep[:mt], C[mt * g:t + 1]], 0)          # representatives, then the tokens after them
        pos = np.concatenate([kr_rep[:mt], KR[mt * g:t + 1]], 0)
        for h in range(H):
            keys = np.concatenate([sem @ wuk[h], pos], 1)               # k = [c W^UK, k^R]   (un-absorbed, per head)
            vals = sem @ wuv[h]                                         # v = c W^UV
            lg = keys @ np.concatenate([qn[t, h], qr[t, h]]) * Hh.f32(scale)
            e = np.exp(lg - lg.max())
            ref[x, h] = (e / e.sum()) @ vals
    got = out_v[0][torch.tensor(rows, device=DEV)]
    # the device saw q_latent rounded to bf16 (logits shift by ~3e-3), then two bf16 roundings (latent output,
    # projected output) on values of unit scale
    st = Hh.check_outputs(got, ref, "absorbed attention + W^UV vs un-absorbed attention")
    assert st["max_abs"] < 2e-2


@pytest.mark.parametrize("kind", ["mla_generic", "mla_fast", "gqa"])
def test_ragged_batch_equals_one_call_per_sequence_and_the_oracle(B, kind):
    # Alg. 1 takes one L per sequence: four sequences of 1, 50, 777 and 2000 tokens packed into one call (no group,
    # no group, 40-odd groups, 100-odd groups; the last tile of one sequence overlaps the first rows of the next)
    # must give, bit for bit, what four single calls give, and match the oracle sequence by sequence.
    lens = [1, 50, 777, 2000]
    if kind == "gqa":
        base = I.scaled(I.CONFIGS["gqa_64k"], n_q_heads=8, n_kv_heads=2, group_size=16, window=40, n_needles=2)
        make = I.make_gqa_inputs
        names = dict(q_sem=None, q_pos="q", kv_sem="v", kv_pos="k")
    else:
        g, w = (16, 64) if kind == "mla_generic" else (64, 128)
        base = I.scaled(I.CONFIGS["mla_1k"], n_q_heads=16, group_size=g, window=w, n_needles=2)
        make = I.make_mla_inputs
        names = dict(q_sem="q_sem", q_pos="q_pos", kv_sem="ckv", kv_pos="kr")
    g, w = base.group_size, base.window
    seqs = [make(I.scaled(base, seq_len=L), "cpu", batch_index=b) for b, L in enumerate(lens)]
    packed = {k: torch.cat([s_[k] for s_ in seqs]).to(DEV) for k in seqs[0]}
    arg = lambda d, key: None if names[key] is None else d[names[key]]
    p = B.params_from_config(I.scaled(base, seq_len=max(lens)), batch=len(lens))
    cond = B.condense_varlen(p, lens, arg(packed, "q_sem"), arg(packed, "q_pos"), arg(packed, "kv_sem"), arg(packed, "kv_pos"))
    out, lse = B.prefill_attention_varlen(p, lens, arg(packed, "q_sem"), arg(packed, "q_pos"), arg(packed, "kv_sem"),
                                          arg(packed, "kv_pos"), cond["cache_sem"], cond["cache_pos"], want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    tok, cro, gro = cond["token_offsets"], cond["cache_row_offsets"], cond["group_offsets"]
    assert tok == [0, 1, 51, 828, 2828]
    for b, L in enumerate(lens):
        d = {k: v.to(DEV) for k, v in seqs[b].items()}
        p1 = B.params_from_config(I.scaled(base, seq_len=L), batch=1)
        n = min(L, g)
        qs = arg(d, "q_sem")
        one = B.condense(p1, None if qs is None else qs[L - n:], arg(d, "q_pos")[L - n:], arg(d, "kv_sem"), arg(d, "kv_pos"))
        o1, l1 = B.prefill_attention(p1, qs, arg(d, "q_pos"), arg(d, "kv_sem"), arg(d, "kv_pos"), one["cache_sem"],
                                     one["cache_pos"], want_lse=True)
        m, k = one["m"], one["k"]
        assert (cro[b + 1] - cro[b], gro[b + 1] - gro[b]) == (m + k, m)
        assert torch.equal(Hh.bits_t(cond["cache_sem"][cro[b]:cro[b + 1]]), Hh.bits_t(one["cache_sem"][0]))
        assert torch.equal(Hh.bits_t(cond["cache_pos"][cro[b]:cro[b + 1]]), Hh.bits_t(one["cache_pos"][0]))
        if m:
            assert torch.equal(cond["anchor_idx"][gro[b]:gro[b + 1]], one["anchor_idx"][0])
        assert torch.equal(Hh.bits_t(out[tok[b]:tok[b + 1]]), Hh.bits_t(o1[0])), f"sequence {b}"
        assert torch.equal(lse[tok[b]:tok[b + 1]], l1[0])
        rows = np.arange(L) if L <= 777 else Hh.sample_positions(L, g, w, n_uniform=40, seed=b)
        if kind == "gqa":
            ref = Hh.oracle_gqa(seqs[b], g, w, base.softmax_scale, rows=rows)
        else:
            ref = Hh.oracle_mla(seqs[b], g, w, base.softmax_scale, rows=rows)
        piece = dict(m=m, k=k, cache_sem=cond["cache_sem"][cro[b]:cro[b + 1]], cache_pos=cond["cache_pos"][cro[b]:cro[b + 1]],
                     anchor_idx=cond["anchor_idx"][gro[b]:gro[b + 1]])
        Hh.check_condense(piece, ref["cond"], kind="gqa" if kind == "gqa" else "mla")
        Hh.check_outputs(out[tok[b]:tok[b + 1]][torch.from_numpy(rows).to(DEV)], ref, f"ragged {kind} sequence {b}")


@pytest.mark.parametrize("nb,H,cap", [(1, 128, 5057), (8, 128, 2100), (3, 256, 900), (5, 16, 700), (37, 128, 600), (64, 128, 300)])
def test_decode_key_ranges_split_over_cta_pairs_match_oracle(B, nb, H, cap):
    # Few sequences: the key tiles of all sequences are cut into equal ranges, one per CTA pair, and a sequence's
    # partial results are merged by a second kernel (one sequence of 40 tiles becomes 40 single-tile ranges; eight
    # ragged ones share ranges; two head blocks per sequence; 16 heads use an eighth of a tile's rows; 37 sequences
    # are the most that are still cut on 74 resident pairs).  64 sequences: whole sequences per work item, no merge.
    # Ragged counts, an empty cache, lse.
    gen = torch.Generator().manual_seed(nb * 1000 + H)
    cache_sem = torch.randn((nb, cap, 1, 512), generator=gen).bfloat16()
    cache_pos = torch.randn((nb, cap, 1, 64), generator=gen).bfloat16()
    q_sem = torch.randn((nb, H, 512), generator=gen).bfloat16()
    q_pos = torch.randn((nb, H, 64), generator=gen).bfloat16()
    rows = torch.randint(1, cap + 1, (nb,), generator=gen, dtype=torch.int32)
    rows[0] = cap
    if nb > 2:
        rows[1] = 0
        rows[2] = 129
    n_rep = 33
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=nb, seq_len=4096, n_q_heads=H)
    p = B.params_from_config(cfg, batch=nb)
    out, lse = B.decode_attention(p, q_sem.to(DEV), q_pos.to(DEV), cache_sem.to(DEV), cache_pos.to(DEV), rows.to(DEV), n_rep,
                                  want_lse=True)
    out2, lse2 = B.decode_attention(p, q_sem.to(DEV), q_pos.to(DEV), cache_sem.to(DEV), cache_pos.to(DEV), rows.to(DEV), n_rep,
                                    want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    assert torch.equal(Hh.bits_t(out), Hh.bits_t(out2)) and torch.equal(lse, lse2)      # fixed merge order: reproducible
    for b in sorted(set(list(range(0, nb, max(1, nb // 6))) + [0, min(1, nb - 1), min(2, nb - 1)])):
        n = int(rows[b])
        if n == 0:
            assert torch.count_nonzero(out[b]) == 0
            assert torch.isinf(lse[b]).all() and (lse[b] < 0).all()
            continue
        cs = O.bits_to_f64(Hh.bits(cache_sem[b, :n, 0]))
        cp = O.bits_to_f64(Hh.bits(cache_pos[b, :n, 0]))
        ro, rl = O.mla_decode(O.torch_bf16_to_f64(q_sem[b]), O.torch_bf16_to_f64(q_pos[b]), cs, cp, min(n_rep, n),
                              Hh.f32(cfg.softmax_scale), 0.0)
        Hh.check_outputs(out[b], ro, f"split decode nb={nb} H={H} seq {b} rows {n}")
        np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)


def test_gqa_prefill_is_bit_reproducible_across_launches(B):
    # Two softmax groups and the MMA warp of a CTA run at their own pace; every hand-off between them must be an
    # ordering, not a coincidence of timing: four launches on the same inputs agree in every bit (sequence long
    # enough for ~70 key tiles per block, 4096 CTAs in all).
    cfg = I.scaled(I.CONFIGS["gqa_64k"], seq_len=8192, group_size=64, window=4096)
    d = to_dev(I.make_gqa_inputs(cfg, "cpu"))
    L, g = cfg.seq_len, cfg.group_size
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, None, d["q"][L - g:], d["v"], d["k"])
    first = None
    for _ in range(4):
        out, lse = B.prefill_attention(p, None, d["q"], d["v"], d["k"], cond["cache_sem"], cond["cache_pos"], want_lse=True)
        torch.cuda.synchronize()
        if first is None:
            first = (out.clone(), lse.clone())
        else:
            assert torch.equal(Hh.bits_t(out), Hh.bits_t(first[0])) and torch.equal(lse, first[1])
    assert B.lca_last_device_status() == 0


def test_random_shapes_match_oracle(B):
    # Seeded sweep over shapes the other cases do not list: lengths around tile and group boundaries, group sizes that
    # do not divide anything, windows from 0 to beyond the sequence, head counts of every tile split, summary lengths,
    # bias on and off; MLA and GQA; prefill on every row and a decode of the last token against the resulting cache.
    rng = np.random.default_rng(2604)
    for case in range(14):
        mla = case % 2 == 0
        L = int(rng.choice([1, 2, 63, 64, 65, 127, 128, 129, 200, 255, 257, 400, 511, 640]))
        g = int(rng.choice([1, 2, 3, 8, 16, 33, 64]))
        w = int(rng.choice([0, 1, 7, 32, 64, 100, 300, 1000]))
        ns = int(rng.choice([0, 1, 5, 64]))
        bias = float(rng.choice([0.0, 0.5]))
        if mla:
            H = int(rng.choice([1, 2, 4, 8, 16, 32, 64, 128]))
            cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=L, n_q_heads=H, group_size=g, window=w, n_needles=min(3, L))
            inp = I.make_mla_inputs(cfg, "cpu")
            d = to_dev(inp)
            p = B.params_from_config(cfg, batch=1, n_summary_q=ns, rep_logit_bias=bias)
            n = min(L, ns if ns > 0 else g)
            cond = B.condense(p, d["q_sem"][L - n:], d["q_pos"][L - n:], d["ckv"], d["kr"])
            out, lse = B.prefill_attention(p, d["q_sem"], d["q_pos"], d["ckv"], d["kr"], cond["cache_sem"], cond["cache_pos"], want_lse=True)
            rows = torch.tensor([cond["m"] + cond["k"]], dtype=torch.int32, device=DEV)
            dout, _ = B.decode_attention(p, d["q_sem"][L - 1].contiguous()[None], d["q_pos"][L - 1].contiguous()[None],
                                         cond["cache_sem"], cond["cache_pos"], rows, cond["m"])
            ref = Hh.oracle_mla(inp, g, w, cfg.softmax_scale, rows=np.arange(L), n_summary=ns, rep_logit_bias=bias)
            kind = "mla"
        else:
            Hkv = int(rng.choice([1, 2, 4]))
            Hq = Hkv * int(rng.choice([1, 2, 4, 8]))
            cfg = I.scaled(I.CONFIGS["gqa_64k"], seq_len=L, n_q_heads=Hq, n_kv_heads=Hkv, group_size=g, window=w, n_needles=min(3, L))
            inp = I.make_gqa_inputs(cfg, "cpu")
            d = to_dev(inp)
            p = B.params_from_config(cfg, batch=1, n_summary_q=ns, rep_logit_bias=bias)
            n = min(L, ns if ns > 0 else g)
            cond = B.condense(p, None, d["q"][L - n:], d["v"], d["k"])
            out, lse = B.prefill_attention(p, None, d["q"], d["v"], d["k"], cond["cache_sem"], cond["cache_pos"], want_lse=True)
            rows = torch.tensor([cond["m"] + cond["k"]], dtype=torch.int32, device=DEV)
            dout, _ = B.decode_attention(p, None, d["q"][L - 1].contiguous()[None], cond["cache_sem"], cond["cache_pos"], rows, cond["m"])
            ref = Hh.oracle_gqa(inp, g, w, cfg.softmax_scale, rows=np.arange(L), n_summary=ns, rep_logit_bias=bias)
            kind = "gqa"
        torch.cuda.synchronize()
        what = f"case {case} {kind} L={L} g={g} w={w} ns={ns} bias={bias} heads={cfg.n_q_heads}/{cfg.n_kv_heads}"
        assert B.lca_last_device_status() == 0, what
        Hh.check_condense(one_seq(cond), ref["cond"], kind=kind)
        Hh.check_outputs(out[0], ref, what)
        np.testing.assert_allclose(lse[0].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4, err_msg=what)
        # decoding the last token against the final cache is the last prefill row (Sec. 4.3)
        Hh.check_outputs(dout[0], ref["out"][-1], what + " decode", vmax=ref["vmax"])


# ------------------------------------------------------------------ ring layout of the decode cache
def _ring_states(g, w, cap, specs, d_sem, d_pos, gen, heads=None):
    """Random packed caches with (n_rep, uncondensed tokens) per sequence -> (packed sem, pos [B, cap_packed, ...],
    packed_rows, n_rep).  heads = None: one KV stream ([.., 1, d]); else [.., heads, d]."""
    hk = 1 if heads is None else heads
    cap_packed = max(r + c for r, c in specs) + 1
    sem = torch.zeros((len(specs), cap_packed, hk, d_sem), dtype=torch.bfloat16)
    pos = torch.zeros((len(specs), cap_packed, hk, d_pos), dtype=torch.bfloat16)
    for b, (r, c) in enumerate(specs):
        sem[b, :r + c] = torch.randn((r + c, hk, d_sem), generator=gen).bfloat16()
        pos[b, :r + c] = torch.randn((r + c, hk, d_pos), generator=gen).bfloat16()
    return sem, pos, [r + c for r, c in specs], [r for r, _ in specs]


@pytest.mark.parametrize("impl,bias", [(0, 0.0), (0, math.log(16.0)), (1, 0.3)])
def test_ring_cache_streaming_matches_oracle_over_many_decode_steps(B, impl, bias):
    # Ring of R = w + g = 192 rows (one and a half key tiles, so the representatives start in the middle of a tile).
    # Three sequences in different phases, one of them so short that its ring has not wrapped; more than two trips
    # round the ring.  Every step: append the token at its ring row, decode (device against the oracle on the rows
    # that take part), update (device against the oracle: only the new representative's row may change).
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=3, seq_len=0, n_q_heads=16, group_size=16, window=176)
    g, w, H, Bsz = cfg.group_size, cfg.window, cfg.n_q_heads, 3
    R = w + g
    steps = 2 * R + g + 7
    cap = R + 8 + steps // g + 4
    gen = torch.Generator().manual_seed(29)
    specs = [(3, w + g - 1), (5, w + 3), (0, 9)]                   # (representatives, uncondensed tokens)
    psem, ppos, prow, prep = _ring_states(g, w, cap, specs, 512, 64, gen)
    p = B.params_from_config(cfg, batch=Bsz, rep_logit_bias=bias)
    d_rep = torch.tensor(prep, dtype=torch.int32, device=DEV)
    d_sem, d_pos, d_tok = B.ring_from_packed(p, psem.to(DEV), ppos.to(DEV), torch.tensor(prow, dtype=torch.int32, device=DEV),
                                             d_rep, cap)
    o_sem, o_pos, o_tok, o_rep = [], [], [], list(prep)
    for b in range(Bsz):
        s, q, n = O.ring_from_packed(Hh.bits(psem[b, :, 0]), Hh.bits(ppos[b, :, 0]), prep[b], prow[b], g, w, cap)
        o_sem.append(s); o_pos.append(q); o_tok.append(n)
        assert np.array_equal(Hh.bits(d_sem[b, :, 0]), s) and np.array_equal(Hh.bits(d_pos[b, :, 0]), q)
    assert d_tok.cpu().tolist() == o_tok
    scale = Hh.f32(cfg.softmax_scale)
    prev = B.lca_set_attention_impl(impl)
    n_updates = 0
    try:
        for step in range(steps):
            new_sem = torch.randn((Bsz, 512), generator=gen).bfloat16()
            new_pos = torch.randn((Bsz, 64), generator=gen).bfloat16()
            for b in range(Bsz):                       # the caller writes the new token at its ring row and counts it
                d_sem[b, o_tok[b] % R, 0] = new_sem[b].to(DEV)
                d_pos[b, o_tok[b] % R, 0] = new_pos[b].to(DEV)
                o_sem[b][o_tok[b] % R] = Hh.bits(new_sem[b])
                o_pos[b][o_tok[b] % R] = Hh.bits(new_pos[b])
                o_tok[b] += 1
            d_tok += 1
            if step % 3 == 0 or step >= steps - 40:
                q_sem = torch.randn((Bsz, H, 512), generator=gen).bfloat16()
                q_pos = torch.randn((Bsz, H, 64), generator=gen).bfloat16()
                out, lse = B.decode_attention_ring(p, q_sem.to(DEV), q_pos.to(DEV), d_sem, d_pos, d_rep, d_tok, want_lse=True)
                torch.cuda.synchronize()
                assert B.lca_last_device_status() == 0
                for b in range(Bsz):
                    cs, cp, n_rows = O.ring_to_packed(o_sem[b], o_pos[b], o_rep[b], o_tok[b], g, w)
                    ro, rl = O.mla_decode(O.torch_bf16_to_f64(q_sem[b]), O.torch_bf16_to_f64(q_pos[b]), O.bits_to_f64(cs),
                                          O.bits_to_f64(cp), o_rep[b], scale, bias)
                    Hh.check_outputs(out[b], ro, f"ring decode step {step} seq {b}")
                    np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)
            q_tail_sem = torch.randn((Bsz, g, H, 512), generator=gen).bfloat16()
            q_tail_pos = torch.randn((Bsz, g, H, 64), generator=gen).bfloat16()
            anchor = B.decode_update_ring(p, q_tail_sem.to(DEV), q_tail_pos.to(DEV), d_sem, d_pos, d_rep, d_tok)
            torch.cuda.synchronize()
            for b in range(Bsz):
                qbar = O.mla_summary_query(O.torch_bf16_to_f64(q_tail_sem[b]), O.torch_bf16_to_f64(q_tail_pos[b]))
                s2, p2, nr, ia = O.mla_decode_update_ring(o_sem[b], o_pos[b], o_rep[b], o_tok[b], qbar, g, w, scale)
                assert int(anchor[b, 0]) == ia
                if ia >= 0:
                    n_updates += 1
                    got_sem, got_pos = Hh.bits(d_sem[b, :, 0]), Hh.bits(d_pos[b, :, 0])
                    row = R + o_rep[b]
                    assert np.array_equal(got_pos, p2)                                   # anchor row: a bit copy; nothing else moved
                    assert (Hh.bf16_ulp_distance(got_sem[row], s2[row]) <= 1).all()      # representative: fp32 pooling
                    s2[row] = got_sem[row]                                               # carry the device's rounding forward
                    assert np.array_equal(got_sem, s2)
                o_sem[b], o_pos[b], o_rep[b] = s2, p2, nr
            assert d_rep.cpu().tolist() == o_rep and d_tok.cpu().tolist() == o_tok
    finally:
        B.lca_set_attention_impl(prev)
    assert n_updates >= 3 * (steps // g) - 12


def test_ring_decode_without_key_range_split_and_full_representative_region(B):
    # 40 sequences x 16 heads: more units than half the CTA pairs, so every unit is one work item (no partial results).
    # States: ring exactly full, one token after an update (g - 1 stale rows), ring not wrapped, empty sequence.
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=40, seq_len=0, n_q_heads=16, group_size=32, window=224)
    g, w, H, Bsz = cfg.group_size, cfg.window, cfg.n_q_heads, 40
    R = w + g
    gen = torch.Generator().manual_seed(31)
    specs = []
    for b in range(Bsz):
        kind = b % 5
        specs.append([(b % 7 + 1, R), (b % 9 + 1, w + 1), (0, 1 + (b * 13) % (R - 1)), (0, 0), (b % 11 + 2, w + g // 2)][kind])
    cap = R + 16
    psem, ppos, prow, prep = _ring_states(g, w, cap, specs, 512, 64, gen)
    p = B.params_from_config(cfg, batch=Bsz, rep_logit_bias=0.5)
    d_rep = torch.tensor(prep, dtype=torch.int32, device=DEV)
    d_sem, d_pos, d_tok = B.ring_from_packed(p, psem.to(DEV), ppos.to(DEV), torch.tensor(prow, dtype=torch.int32, device=DEV),
                                             d_rep, cap)
    q_sem = torch.randn((Bsz, H, 512), generator=gen).bfloat16()
    q_pos = torch.randn((Bsz, H, 64), generator=gen).bfloat16()
    out, lse = B.decode_attention_ring(p, q_sem.to(DEV), q_pos.to(DEV), d_sem, d_pos, d_rep, d_tok, want_lse=True)
    torch.cuda.synchronize()
    assert B.lca_last_device_status() == 0
    tok = d_tok.cpu().tolist()
    for b in range(Bsz):
        r, c = specs[b]
        assert tok[b] == r * g + c
        if r + c == 0:
            assert float(out[b].abs().max()) == 0.0 and bool(torch.isinf(lse[b]).all())
            continue
        cs, cp, n_rows = O.ring_to_packed(Hh.bits(d_sem[b, :, 0]), Hh.bits(d_pos[b, :, 0]), r, tok[b], g, w)
        assert n_rows == r + c
        assert np.array_equal(cs, Hh.bits(psem[b, :r + c, 0])) and np.array_equal(cp, Hh.bits(ppos[b, :r + c, 0]))
        ro, rl = O.mla_decode(O.torch_bf16_to_f64(q_sem[b]), O.torch_bf16_to_f64(q_pos[b]), O.bits_to_f64(cs), O.bits_to_f64(cp),
                              r, Hh.f32(cfg.softmax_scale), 0.5)
        Hh.check_outputs(out[b], ro, f"ring decode seq {b}")
        np.testing.assert_allclose(lse[b].cpu().numpy(), rl, atol=2e-3, rtol=1e-4)


def test_gqa_ring_decode_matches_oracle(B):
    # GQA cache in the ring layout (one ring per KV head, same rows): the one-tile tensor-core kernel and the scalar kernel
    cfg = I.scaled(I.CONFIGS["gqa_64k"], batch=4, seq_len=0, n_q_heads=32, n_kv_heads=8, group_size=64, window=192)
    g, w, Hq, Hkv, d = cfg.group_size, cfg.window, cfg.n_q_heads, cfg.n_kv_heads, cfg.d_sem
    R = w + g
    gen = torch.Generator().manual_seed(37)
    specs = [(6, R), (2, w + 5), (0, 77), (9, w + g - 1)]
    cap = R + 12
    pv, pk, prow, prep = _ring_states(g, w, cap, specs, d, d, gen, heads=Hkv)
    p = B.params_from_config(cfg, batch=4, rep_logit_bias=0.25)
    d_rep = torch.tensor(prep, dtype=torch.int32, device=DEV)
    ring_v, ring_k, d_tok = B.ring_from_packed(p, pv.to(DEV), pk.to(DEV), torch.tensor(prow, dtype=torch.int32, device=DEV), d_rep, cap)
    q = torch.randn((4, Hq, d), generator=gen).bfloat16()
    refs = []
    for b, (r, c) in enumerate(specs):
        refs.append(O.gqa_decode(O.torch_bf16_to_f64(q[b]), O.bits_to_f64(Hh.bits(pk[b, :r + c])), O.bits_to_f64(Hh.bits(pv[b, :r + c])),
                                 r, Hh.f32(cfg.softmax_scale), 0.25))
    for impl in (0, 1):
        prev = B.lca_set_attention_impl(impl)
        try:
            out, lse = B.decode_attention_ring(p, None, q.to(DEV), ring_v, ring_k, d_rep, d_tok, want_lse=True)
        finally:
            B.lca_set_attention_impl(prev)
        torch.cuda.synchronize()
        assert B.lca_last_device_status() == 0
        for b in range(4):
            Hh.check_outputs(out[b], refs[b][0], f"gqa ring decode seq {b} impl {impl}")
            np.testing.assert_allclose(lse[b].cpu().numpy(), refs[b][1], atol=2e-3, rtol=1e-4)


def test_ring_cache_step_update_with_running_summary_query_matches_oracle(B):
    # One call per decode step: the step's queries go into the running sum, sequences that are due are condensed with
    # the mean of everything summed since their previous update.  Oracle: the same queries collected per sequence and
    # averaged by mla_summary_query.  The sequences are in different phases, so the first updates use fewer than g queries.
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=3, seq_len=0, n_q_heads=16, group_size=16, window=48)
    g, w, H, Bsz = cfg.group_size, cfg.window, cfg.n_q_heads, 3
    R = w + g
    steps = 3 * g + 5
    cap = R + 8 + steps // g + 2
    gen = torch.Generator().manual_seed(41)
    specs = [(2, w + g - 3), (4, w + 1), (0, 20)]
    psem, ppos, prow, prep = _ring_states(g, w, cap, specs, 512, 64, gen)
    p = B.params_from_config(cfg, batch=Bsz)
    d_rep = torch.tensor(prep, dtype=torch.int32, device=DEV)
    d_sem, d_pos, d_tok = B.ring_from_packed(p, psem.to(DEV), ppos.to(DEV), torch.tensor(prow, dtype=torch.int32, device=DEV),
                                             d_rep, cap)
    o_sem = [Hh.bits(d_sem[b, :, 0]) for b in range(Bsz)]
    o_pos = [Hh.bits(d_pos[b, :, 0]) for b in range(Bsz)]
    o_tok, o_rep = d_tok.cpu().tolist(), list(prep)
    qsum = torch.zeros((Bsz, 1, 576), dtype=torch.float64, device=DEV)
    qcount = torch.zeros((Bsz,), dtype=torch.int32, device=DEV)
    seen = [[] for _ in range(Bsz)]
    scale = Hh.f32(cfg.softmax_scale)
    n_updates = 0
    for step in range(steps):
        new_sem = torch.randn((Bsz, 512), generator=gen).bfloat16()
        new_pos = torch.randn((Bsz, 64), generator=gen).bfloat16()
        for b in range(Bsz):
            d_sem[b, o_tok[b] % R, 0] = new_sem[b].to(DEV)
            d_pos[b, o_tok[b] % R, 0] = new_pos[b].to(DEV)
            o_sem[b][o_tok[b] % R] = Hh.bits(new_sem[b])
            o_pos[b][o_tok[b] % R] = Hh.bits(new_pos[b])
            o_tok[b] += 1
        d_tok += 1
        q_sem = torch.randn((Bsz, H, 512), generator=gen).bfloat16()
        q_pos = torch.randn((Bsz, H, 64), generator=gen).bfloat16()
        anchor = B.decode_step_update_ring(p, q_sem.to(DEV), q_pos.to(DEV), qsum, qcount, d_sem, d_pos, d_rep, d_tok)
        torch.cuda.synchronize()
        for b in range(Bsz):
            seen[b].append((q_sem[b], q_pos[b]))
            qbar = O.mla_summary_query(O.torch_bf16_to_f64(torch.stack([s for s, _ in seen[b]])),
                                       O.torch_bf16_to_f64(torch.stack([q for _, q in seen[b]])))
            s2, p2, nr, ia = O.mla_decode_update_ring(o_sem[b], o_pos[b], o_rep[b], o_tok[b], qbar, g, w, scale)
            assert int(anchor[b, 0]) == ia
            if ia >= 0:
                n_updates += 1
                seen[b] = []
                got_sem, got_pos = Hh.bits(d_sem[b, :, 0]), Hh.bits(d_pos[b, :, 0])
                row = R + o_rep[b]
                assert np.array_equal(got_pos, p2)
                assert (Hh.bf16_ulp_distance(got_sem[row], s2[row]) <= 1).all()
                s2[row] = got_sem[row]
                assert np.array_equal(got_sem, s2)
                assert float(qsum[b].abs().max()) == 0.0
            o_sem[b], o_pos[b], o_rep[b] = s2, p2, nr
        assert d_rep.cpu().tolist() == o_rep and qcount.cpu().tolist() == [len(x) for x in seen]
    assert n_updates >= 8


def test_gqa_ring_cache_update_matches_oracle(B):
    # GQA variant of the online update (pool V, select K, per KV head) on the ring layout: query tails, then the per-step
    # form with the running summary query; three sequences in different phases, g + 3 steps.
    cfg = I.scaled(I.CONFIGS["gqa_64k"], batch=3, seq_len=0, n_q_heads=16, n_kv_heads=4, group_size=16, window=48)
    g, w, Hq, Hkv, d, Bsz = cfg.group_size, cfg.window, cfg.n_q_heads, cfg.n_kv_heads, cfg.d_sem, 3
    R = w + g
    steps = g + 3
    cap = R + 8
    gen = torch.Generator().manual_seed(43)
    specs = [(2, w + g - 2), (4, w + 1), (0, w + g - 1)]
    pv, pk, prow, prep = _ring_states(g, w, cap, specs, d, d, gen, heads=Hkv)
    p = B.params_from_config(cfg, batch=Bsz)
    scale = Hh.f32(cfg.softmax_scale)
    for form in ("tails", "step"):
        d_rep = torch.tensor(prep, dtype=torch.int32, device=DEV)
        ring_v, ring_k, d_tok = B.ring_from_packed(p, pv.to(DEV), pk.to(DEV), torch.tensor(prow, dtype=torch.int32, device=DEV), d_rep, cap)
        o_k = [Hh.bits(ring_k[b]) for b in range(Bsz)]
        o_v = [Hh.bits(ring_v[b]) for b in range(Bsz)]
        o_tok, o_rep = d_tok.cpu().tolist(), list(prep)
        qsum = torch.zeros((Bsz, Hkv, d), dtype=torch.float64, device=DEV)
        qcount = torch.zeros((Bsz,), dtype=torch.int32, device=DEV)
        seen = [[] for _ in range(Bsz)]
        n_updates = 0
        for step in range(steps):
            new_k = torch.randn((Bsz, Hkv, d), generator=gen).bfloat16()
            new_v = torch.randn((Bsz, Hkv, d), generator=gen).bfloat16()
            for b in range(Bsz):
                ring_k[b, o_tok[b] % R] = new_k[b].to(DEV)
                ring_v[b, o_tok[b] % R] = new_v[b].to(DEV)
                o_k[b][o_tok[b] % R] = Hh.bits(new_k[b])
                o_v[b][o_tok[b] % R] = Hh.bits(new_v[b])
                o_tok[b] += 1
            d_tok += 1
            if form == "tails":
                q_tail = torch.randn((Bsz, g, Hq, d), generator=gen).bfloat16()
                anchor = B.decode_update_ring(p, None, q_tail.to(DEV), ring_v, ring_k, d_rep, d_tok)
            else:
                q_now = torch.randn((Bsz, Hq, d), generator=gen).bfloat16()
                anchor = B.decode_step_update_ring(p, None, q_now.to(DEV), qsum, qcount, ring_v, ring_k, d_rep, d_tok)
            torch.cuda.synchronize()
            for b in range(Bsz):
                if form == "tails":
                    qbar = O.gqa_summary_query(O.torch_bf16_to_f64(q_tail[b]), Hkv)
                else:
                    seen[b].append(q_now[b])
                    qbar = O.gqa_summary_query(O.torch_bf16_to_f64(torch.stack(seen[b])), Hkv)
                k2, v2, nr, anc = O.gqa_decode_update_ring(o_k[b], o_v[b], o_rep[b], o_tok[b], qbar, g, w, scale)
                if anc is None:
                    assert (anchor[b].cpu().numpy() == -1).all()
                else:
                    n_updates += 1
                    seen[b] = []
                    assert np.array_equal(anchor[b].cpu().numpy(), anc)
                    got_k, got_v = Hh.bits(ring_k[b]), Hh.bits(ring_v[b])
                    row = R + o_rep[b]
                    assert np.array_equal(got_k, k2)                                     # selected keys: bit copies, per head
                    assert (Hh.bf16_ulp_distance(got_v[row], v2[row]) <= 1).all()        # pooled values: fp32 pooling
                    v2[row] = got_v[row]
                    assert np.array_equal(got_v, v2)
                o_k[b], o_v[b], o_rep[b] = k2, v2, nr
            assert d_rep.cpu().tolist() == o_rep
        assert n_updates >= 3


def test_gqa_packed_cache_update_matches_oracle(B):
    # lca_decode_update (packed layout, the window moves up) for the GQA variant: one call on three sequences, two of them
    # due.  Expected state: the oracle's ring update read back in packed order (the two layouts hold the same rows).
    cfg = I.scaled(I.CONFIGS["gqa_64k"], batch=3, seq_len=0, n_q_heads=16, n_kv_heads=4, group_size=16, window=48)
    g, w, Hq, Hkv, d, Bsz = cfg.group_size, cfg.window, cfg.n_q_heads, cfg.n_kv_heads, cfg.d_sem, 3
    R = w + g
    gen = torch.Generator().manual_seed(47)
    specs = [(2, R), (4, w + 5), (0, R)]
    cap = R + 8
    pv, pk, prow, prep = _ring_states(g, w, cap, specs, d, d, gen, heads=Hkv)
    capacity = pv.shape[1]
    p = B.params_from_config(cfg, batch=Bsz)
    d_v, d_k = pv.to(DEV), pk.to(DEV)
    d_rep = torch.tensor(prep, dtype=torch.int32, device=DEV)
    d_rows = torch.tensor(prow, dtype=torch.int32, device=DEV)
    q_tail = torch.randn((Bsz, g, Hq, d), generator=gen).bfloat16()
    anchor = B.decode_update(p, None, q_tail.to(DEV), d_v, d_k, d_rep, d_rows)
    torch.cuda.synchronize()
    for b, (r, c) in enumerate(specs):
        rk, rv, n_tok = O.ring_from_packed(Hh.bits(pk[b]), Hh.bits(pv[b]), r, r + c, g, w, cap)
        qbar = O.gqa_summary_query(O.torch_bf16_to_f64(q_tail[b]), Hkv)
        k2, v2, nr, anc = O.gqa_decode_update_ring(rk, rv, r, n_tok, qbar, g, w, Hh.f32(cfg.softmax_scale))
        ek, ev, n_rows = O.ring_to_packed(k2, v2, nr, n_tok, g, w)
        assert int(d_rep[b]) == nr and int(d_rows[b]) == n_rows and (anc is None) == (c < R)
        got_k, got_v = Hh.bits(d_k[b, :n_rows]), Hh.bits(d_v[b, :n_rows])
        if anc is None:
            assert (anchor[b].cpu().numpy() == -1).all()
        else:
            assert np.array_equal(anchor[b].cpu().numpy(), anc)
            assert (Hh.bf16_ulp_distance(got_v[nr - 1], ev[nr - 1]) <= 1).all()
            ev[nr - 1] = got_v[nr - 1]
        assert np.array_equal(got_k, ek) and np.array_equal(got_v, ev)
    assert capacity >= max(prow)


@pytest.mark.parametrize("kind", ["mla_dc128", "gqa_d64"])
def test_smaller_head_shapes_on_the_scalar_kernel_match_oracle(B, kind):
    # Shapes without a tensor-core kernel (MLA with a 128-wide latent, GQA with 64-wide heads): generic condensation
    # kernel and the scalar attention kernel; prefill on every row, decode over the packed cache and over the ring layout.
    g, w, L = 16, 48, 333
    if kind == "mla_dc128":
        cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=L, n_q_heads=6, group_size=g, window=w, d_sem=128, n_needles=2)
        inp = I.make_mla_inputs(cfg, "cpu")
        d = to_dev(inp)
        p = B.params_from_config(cfg, batch=1, rep_logit_bias=0.4)
        cond = B.condense(p, d["q_sem"][L - g:], d["q_pos"][L - g:], d["ckv"], d["kr"])
        out, lse = B.prefill_attention(p, d["q_sem"], d["q_pos"], d["ckv"], d["kr"], cond["cache_sem"], cond["cache_pos"], want_lse=True)
        ref = Hh.oracle_mla(inp, g, w, cfg.softmax_scale, rows=np.arange(L), rep_logit_bias=0.4)
        q_last = (d["q_sem"][L - 1].contiguous()[None], d["q_pos"][L - 1].contiguous()[None])
        ckind = "mla"
    else:
        cfg = I.scaled(I.CONFIGS["gqa_64k"], seq_len=L, n_q_heads=6, n_kv_heads=3, group_size=g, window=w, d_sem=64, n_needles=2)
        inp = I.make_gqa_inputs(cfg, "cpu")
        d = to_dev(inp)
        p = B.params_from_config(cfg, batch=1, rep_logit_bias=0.4)
        cond = B.condense(p, None, d["q"][L - g:], d["v"], d["k"])
        out, lse = B.prefill_attention(p, None, d["q"], d["v"], d["k"], cond["cache_sem"], cond["cache_pos"], want_lse=True)
        ref = Hh.oracle_gqa(inp, g, w, cfg.softmax_scale, rows=np.arange(L), rep_logit_bias=0.4)
        q_last = (None, d["q"][L - 1].contiguous()[None])
        ckind = "gqa"
    torch.cuda.synchronize()
    Hh.check_condense(one_seq(cond), ref["cond"], kind=ckind)
    Hh.check_outputs(out[0], ref, kind)
    np.testing.assert_allclose(lse[0].cpu().numpy(), ref["lse"], atol=2e-3, rtol=1e-4)
    m, k = cond["m"], cond["k"]
    rows = torch.tensor([m + k], dtype=torch.int32, device=DEV)
    dout, _ = B.decode_attention(p, q_last[0], q_last[1], cond["cache_sem"], cond["cache_pos"], rows, m)
    Hh.check_outputs(dout[0], ref["out"][-1], kind + " decode", vmax=ref["vmax"])
    n_rep = torch.tensor([m], dtype=torch.int32, device=DEV)
    ring_sem, ring_pos, n_tok = B.ring_from_packed(p, cond["cache_sem"], cond["cache_pos"], rows, n_rep, w + g + m + 2)
    assert int(n_tok[0]) == L
    rout, _ = B.decode_attention_ring(p, q_last[0], q_last[1], ring_sem, ring_pos, n_rep, n_tok)
    torch.cuda.synchronize()
    Hh.check_outputs(rout[0], ref["out"][-1], kind + " ring decode", vmax=ref["vmax"])


def test_prefill_then_ring_decode_loop_end_to_end(B):
    # The calls composed as a serving loop would use them (MLA shape, tensor-core kernels): condense + prefill of a prompt,
    # the packed cache moved into the ring layout, then decode steps of [append the token, attend, per-step update with the
    # running summary query].  The running sum is primed with the prompt's queries after its last group boundary, so every
    # update uses the last g queries.  Each step against the oracle's streaming state.
    cfg = I.scaled(I.CONFIGS["mla_1k"], seq_len=700, n_q_heads=16, group_size=16, window=48, n_needles=3)
    L, g, w, H = cfg.seq_len, cfg.group_size, cfg.window, cfg.n_q_heads
    R = w + g
    steps = 2 * g + 3
    inp = I.make_mla_inputs(cfg, "cpu")
    d = to_dev(inp)
    p = B.params_from_config(cfg, batch=1)
    scale = Hh.f32(cfg.softmax_scale)
    cond = B.condense(p, d["q_sem"][L - g:], d["q_pos"][L - g:], d["ckv"], d["kr"])
    out, _ = B.prefill_attention(p, d["q_sem"], d["q_pos"], d["ckv"], d["kr"], cond["cache_sem"], cond["cache_pos"])
    ref = Hh.oracle_mla(inp, g, w, cfg.softmax_scale, rows=np.array([L - 1]))
    Hh.check_condense(one_seq(cond), ref["cond"])
    Hh.check_outputs(out[0, L - 1:], ref, "last prefill row")
    m, k = cond["m"], cond["k"]
    n_rep = torch.tensor([m], dtype=torch.int32, device=DEV)
    cap = R + m + steps // g + 2
    ring_sem, ring_pos, n_tok = B.ring_from_packed(p, cond["cache_sem"], cond["cache_pos"],
                                                   torch.tensor([m + k], dtype=torch.int32, device=DEV), n_rep, cap)
    o_sem, o_pos, o_tok = O.ring_from_packed(ref["cond"]["cache_sem_bits"], ref["cond"]["cache_pos_bits"], m, m + k, g, w, cap)
    got = Hh.bits(ring_sem[0, :, 0])
    assert (Hh.bf16_ulp_distance(got[R:R + m], o_sem[R:R + m]) <= 1).all()          # representatives: fp32 pooling on the device
    o_sem[R:R + m] = got[R:R + m]
    assert np.array_equal(got, o_sem) and np.array_equal(Hh.bits(ring_pos[0, :, 0]), o_pos) and int(n_tok[0]) == o_tok == L
    # prime the running sum with the queries of the tokens behind the last group boundary (k - w of them)
    qsum = torch.zeros((1, 1, 576), dtype=torch.float64, device=DEV)
    qcount = torch.zeros((1,), dtype=torch.int32, device=DEV)
    seen = []
    for t in range(L - (k - w), L):
        B.decode_step_update_ring(p, d["q_sem"][t][None].contiguous(), d["q_pos"][t][None].contiguous(), qsum, qcount,
                                  ring_sem, ring_pos, n_rep, n_tok)
        seen.append((inp["q_sem"][t], inp["q_pos"][t]))
    assert int(qcount[0]) == k - w and int(n_rep[0]) == m
    o_rep, gen, n_updates = m, torch.Generator().manual_seed(53), 0
    for step in range(steps):
        new_sem, new_pos = torch.randn((512,), generator=gen).bfloat16(), torch.randn((64,), generator=gen).bfloat16()
        q_sem, q_pos = torch.randn((1, H, 512), generator=gen).bfloat16(), torch.randn((1, H, 64), generator=gen).bfloat16()
        ring_sem[0, o_tok % R, 0], ring_pos[0, o_tok % R, 0] = new_sem.to(DEV), new_pos.to(DEV)
        o_sem[o_tok % R], o_pos[o_tok % R] = Hh.bits(new_sem), Hh.bits(new_pos)
        o_tok += 1
        n_tok += 1
        dout, _ = B.decode_attention_ring(p, q_sem.to(DEV), q_pos.to(DEV), ring_sem, ring_pos, n_rep, n_tok)
        cs, cp, _ = O.ring_to_packed(o_sem, o_pos, o_rep, o_tok, g, w)
        ro, _ = O.mla_decode(O.torch_bf16_to_f64(q_sem[0]), O.torch_bf16_to_f64(q_pos[0]), O.bits_to_f64(cs), O.bits_to_f64(cp), o_rep, scale)
        Hh.check_outputs(dout[0], ro, f"decode step {step}")
        anchor = B.decode_step_update_ring(p, q_sem.to(DEV), q_pos.to(DEV), qsum, qcount, ring_sem, ring_pos, n_rep, n_tok)
        torch.cuda.synchronize()
        seen.append((q_sem[0], q_pos[0]))
        qbar = O.mla_summary_query(O.torch_bf16_to_f64(torch.stack([a for a, _ in seen])), O.torch_bf16_to_f64(torch.stack([c for _, c in seen])))
        s2, p2, nr, ia = O.mla_decode_update_ring(o_sem, o_pos, o_rep, o_tok, qbar, g, w, scale)
        assert int(anchor[0, 0]) == ia
        if ia >= 0:
            assert len(seen) == g                                      # the last g queries
            n_updates, seen = n_updates + 1, []
            got = Hh.bits(ring_sem[0, :, 0])
            assert (Hh.bf16_ulp_distance(got[R + o_rep], s2[R + o_rep]) <= 1).all()
            s2[R + o_rep] = got[R + o_rep]
            assert np.array_equal(got, s2) and np.array_equal(Hh.bits(ring_pos[0, :, 0]), p2)
        o_sem, o_pos, o_rep = s2, p2, nr
        assert int(n_rep[0]) == o_rep
    assert n_updates >= 2 and B.lca_last_device_status() == 0
