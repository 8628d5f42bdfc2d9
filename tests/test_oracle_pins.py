"""Pins for the fp64 CPU oracle: what the mathematics fixes, checked without any GPU.

The paper prints no worked example for this path, so every pin is a brute-force evaluation with
a different structure, a closed form, an invariant, a reduction to a textbook / library routine,
or the paper's own invariant that prefix+suffix scoring equals one-pass scoring (Section 3.1
Phase 2; Section 4.3).
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2608_14498_b200 import workloads as wk

GOLDEN = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")) as fh:
    for line in fh:
        if line.strip() and not line.startswith("#"):
            key, val = line.split()
            GOLDEN[key] = float(val)


def _rand(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


def _batch(lens, hq, hkv, d, seed):
    n = int(np.sum(lens))
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    return _rand((n, hq, d), seed), _rand((n, hkv, d), seed + 1), _rand((n, hkv, d), seed + 2), cu


# ---------------------------------------------------------------- P1 brute force, other structure
def _brute_attention(q, k, v, cu, scale):
    """Whole probability table per (sequence, head) in long double, no max subtraction."""
    hq, hkv = q.shape[1], k.shape[1]
    out = np.zeros(q.shape, dtype=np.longdouble)
    lse = np.zeros(q.shape[:2], dtype=np.longdouble)
    for s in range(len(cu) - 1):
        a, b = int(cu[s]), int(cu[s + 1])
        n = b - a
        for h in range(hq):
            g = h // (hq // hkv)
            qq = q[a:b, h].astype(np.longdouble)
            kk = k[a:b, g].astype(np.longdouble)
            vv = v[a:b, g].astype(np.longdouble)
            e = np.exp(np.einsum("ic,jc->ij", qq, kk) * np.longdouble(scale))
            e = e * np.tril(np.ones((n, n), dtype=np.longdouble))
            z = e.sum(axis=1)
            out[a:b, h] = (e / z[:, None]) @ vv
            lse[a:b, h] = np.log(z)
    return out, lse


@pytest.mark.parametrize("lens,hq,hkv,d", [([8], 2, 1, 4), ([3, 1, 5], 4, 2, 2), ([1], 1, 1, 1), ([7, 8], 6, 2, 3)])
def test_attention_brute_force(lens, hq, hkv, d):
    q, k, v, cu = _batch(lens, hq, hkv, d, seed=3)
    scale = 1.0 / math.sqrt(d)
    ref_o, ref_l = _brute_attention(q, k, v, cu, scale)
    rows = oracle.all_rows(cu, hq)
    o, l = oracle.attn_rows(q, k, v, cu, rows)
    tok = cu[rows[:, 0]] + rows[:, 1]
    np.testing.assert_allclose(o, ref_o[tok, rows[:, 2]].astype(np.float64), rtol=0, atol=1e-12)
    np.testing.assert_allclose(l, ref_l[tok, rows[:, 2]].astype(np.float64), rtol=0, atol=1e-12)


def test_logprob_brute_force():
    n, h, vocab = 6, 5, 8
    hid, w = _rand((n, h), 10), _rand((vocab, h), 11)
    ids = np.arange(n, dtype=np.int32) % vocab
    z = hid.astype(np.longdouble) @ w.astype(np.longdouble).T
    p = np.exp(z) / np.exp(z).sum(axis=1, keepdims=True)
    ref = np.log(p[np.arange(n), ids]).astype(np.float64)
    lp, lse = oracle.logprob_rows(hid, w, ids)
    np.testing.assert_allclose(lp, ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, np.log(np.exp(z).sum(axis=1)).astype(np.float64), rtol=0, atol=1e-12)


# ---------------------------------------------------------------- P2 invariants of the weights
def test_attention_weights_sum_to_one_and_are_causal_and_unpacked():
    lens = [5, 9, 2]
    q, k, _, cu = _batch(lens, 4, 2, 8, seed=20)
    n = int(cu[-1])
    ones = np.ones((n, 2, 8), np.float32)
    rows = oracle.all_rows(cu, 4)
    o, _ = oracle.attn_rows(q, k, ones, cu, rows)
    np.testing.assert_allclose(o, 1.0, rtol=0, atol=1e-14)
    # V[j] = one-hot(global token j): O[i] is then the probability row itself
    q, k, _, cu = _batch(lens, 4, 2, n, seed=21)
    onehot = np.zeros((n, 2, n), np.float32)
    onehot[np.arange(n), :, np.arange(n)] = 1.0
    o, _ = oracle.attn_rows(q, k, onehot, cu, rows)
    assert (o >= 0).all()
    np.testing.assert_allclose(o.sum(axis=1), 1.0, rtol=0, atol=1e-14)
    for r, (s, i, _h) in enumerate(rows):
        allowed = np.zeros(n, bool)
        allowed[cu[s]: cu[s] + i + 1] = True
        assert (o[r][~allowed] == 0.0).all(), "weight on a future token or on another sequence"
        assert (o[r][allowed] > 0.0).all()


# ---------------------------------------------------------------- P3 / P4 closed forms
def test_zero_query_gives_running_mean_and_log_count():
    lens = [8, 3]
    _, k, v, cu = _batch(lens, 2, 2, 4, seed=30)
    q = np.zeros((int(cu[-1]), 2, 4), np.float32)
    rows = oracle.all_rows(cu, 2)
    o, lse = oracle.attn_rows(q, k, v, cu, rows)
    for r, (s, i, h) in enumerate(rows):
        mean = v[cu[s]: cu[s] + i + 1, h].astype(np.float64).mean(axis=0)
        np.testing.assert_allclose(o[r], mean, rtol=0, atol=1e-14)
        assert abs(lse[r] - math.log(i + 1)) < 1e-14
    one = rows[:, 1] == 0
    assert np.abs(lse[one] - GOLDEN["ln_1"]).max() < 1e-15
    assert np.abs(lse[rows[:, 1] == 1] - GOLDEN["ln_2"]).max() < 1e-15
    assert np.abs(lse[rows[:, 1] == 7] - GOLDEN["ln_8"]).max() < 1e-15


def test_first_row_returns_first_value_exactly():
    lens = [4, 6, 1]
    q, k, v, cu = _batch(lens, 6, 3, 5, seed=40)
    rows = np.array([(s, 0, h) for s in range(3) for h in range(6)], np.int32)
    o, lse = oracle.attn_rows(q, k, v, cu, rows)
    for r, (s, _, h) in enumerate(rows):
        assert (o[r] == v[cu[s], h // 2].astype(np.float64)).all()
        dot = float(np.dot(q[cu[s], h].astype(np.float64), k[cu[s], h // 2].astype(np.float64)))
        assert abs(lse[r] - dot / math.sqrt(5)) < 1e-14


@pytest.mark.parametrize("vocab,key", [(4096, "neg_ln_4096"), (152064, "neg_ln_152064")])
def test_zero_weights_give_uniform_logprob(vocab, key):
    hid = _rand((3, 16), 50)
    ids = np.array([0, vocab // 2, vocab - 1], np.int32)
    lp, lse = oracle.logprob_rows(hid, np.zeros((vocab, 16), np.float32), ids)
    assert np.abs(lp - GOLDEN[key]).max() < 1e-13
    assert np.abs(lse + GOLDEN[key]).max() < 1e-13
    lp, _ = oracle.logprob_rows(np.zeros((3, 16), np.float32), _rand((vocab, 16), 51), ids)
    assert np.abs(lp - GOLDEN[key]).max() < 1e-13


def test_probabilities_over_all_targets_sum_to_one():
    vocab, h = 37, 9
    hid = np.repeat(_rand((1, h), 60), vocab, axis=0)
    w = _rand((vocab, h), 61)
    lp, _ = oracle.logprob_rows(hid, w, np.arange(vocab, dtype=np.int32))
    assert abs(np.exp(lp).sum() - 1.0) < 1e-13


def test_out_of_range_target_is_nan():
    lp, _ = oracle.logprob_rows(_rand((2, 4), 1), _rand((8, 4), 2), np.array([8, -1], np.int32))
    assert np.isnan(lp).all()


# ---------------------------------------------------------------- P6 GQA reduces to MHA
def test_gqa_equals_mha_with_replicated_kv_heads():
    lens = [6, 4]
    q, k, v, cu = _batch(lens, 6, 2, 4, seed=70)
    rows = oracle.all_rows(cu, 6)
    o1, l1 = oracle.attn_rows(q, k, v, cu, rows)
    k_rep, v_rep = np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1)  # consecutive q heads share a kv head
    o2, l2 = oracle.attn_rows(q, np.ascontiguousarray(k_rep), np.ascontiguousarray(v_rep), cu, rows)
    assert (o1 == o2).all() and (l1 == l2).all()


# ---------------------------------------------------------------- P7 library special cases
def test_against_torch_fp64_sdpa_and_log_softmax():
    lens = [33, 17, 64]
    hq, hkv, d = 4, 2, 16
    q, k, v, cu = _batch(lens, hq, hkv, d, seed=80)
    rows = oracle.all_rows(cu, hq)
    o, _ = oracle.attn_rows(q, k, v, cu, rows)
    o = o.reshape(int(cu[-1]), hq, d)
    for s in range(len(lens)):
        a, b = int(cu[s]), int(cu[s + 1])
        tq = torch.from_numpy(q[a:b]).double().permute(1, 0, 2)
        tk = torch.from_numpy(np.repeat(k[a:b], hq // hkv, axis=1)).double().permute(1, 0, 2)
        tv = torch.from_numpy(np.repeat(v[a:b], hq // hkv, axis=1)).double().permute(1, 0, 2)
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(1, 0, 2)
        np.testing.assert_allclose(o[a:b], ref.numpy(), rtol=0, atol=1e-10)
    hid, w = _rand((20, 48), 81), _rand((300, 48), 82, 0.3)
    ids = np.random.default_rng(83).integers(0, 300, 20).astype(np.int32)
    ref = torch.log_softmax(torch.from_numpy(hid).double() @ torch.from_numpy(w).double().T, dim=-1)
    ref = ref.gather(1, torch.from_numpy(ids).long()[:, None])[:, 0].numpy()
    lp, _ = oracle.logprob_rows(hid, w, ids)
    np.testing.assert_allclose(lp, ref, rtol=0, atol=1e-10)
    sub = np.array([19, 0, 7], np.int64)
    lp_sub, _ = oracle.logprob_rows(hid, w, ids, rows=sub)
    np.testing.assert_allclose(lp_sub, ref[sub], rtol=0, atol=1e-10)


def test_strided_inputs_and_explicit_scale():
    lens = [9]
    q, k, v, cu = _batch(lens, 2, 1, 4, seed=90)
    wide = np.zeros((9, 5, 4), np.float32)
    wide[:, :2] = q
    rows = oracle.all_rows(cu, 2)
    o1, _ = oracle.attn_rows(q, k, v, cu, rows, scale=0.37)
    o2, _ = oracle.attn_rows(wide[:, :2], k, v, cu, rows, scale=0.37)
    assert (o1 == o2).all()
    ref, _ = _brute_attention(q, k, v, cu, 0.37)
    np.testing.assert_allclose(o1.reshape(9, 2, 4), ref.astype(np.float64), rtol=0, atol=1e-12)


# ---------------------------------------------------------------- dtype handling
def test_bf16_bits_are_promoted_exactly_and_rne_cast_matches_torch():
    x = _rand((4096,), 100)
    x[:6] = [1.00390625, 1.01171875, -1.00390625, 3.3895314e38, 1e-40, 0.0]  # ties, near-overflow, denormal
    bits = wk.f32_to_bf16_bits(x)
    tb = torch.from_numpy(x).to(torch.bfloat16)
    assert (bits == tb.view(torch.int16).numpy().view(np.uint16)).all()
    np.testing.assert_array_equal(wk.bf16_bits_to_f32(bits), tb.float().numpy())
    # oracle fed bf16 bits == oracle fed the same values as float32
    lens = [12]
    q, k, v, cu = _batch(lens, 2, 1, 8, seed=101)
    qb, kb, vb = (wk.f32_to_bf16_bits(t).reshape(t.shape) for t in (q, k, v))
    rows = oracle.all_rows(cu, 2)
    o1, l1 = oracle.attn_rows(qb, kb, vb, cu, rows)
    o2, l2 = oracle.attn_rows(*(wk.bf16_bits_to_f32(t).reshape(t.shape) for t in (qb, kb, vb)), cu, rows)
    assert (o1 == o2).all() and (l1 == l2).all()
    # the cache image of fp32 inputs is the RNE cast (checked against torch's cast)
    table = np.array([[2, 0]], np.int32)
    kc, vc = oracle.cache_image(k, v, cu, table, num_blocks=3)
    ref = torch.from_numpy(k).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert (kc[2, 0, :12] == ref[:12, 0]).all()
    assert (vc[2, 0, :12] == wk.f32_to_bf16_bits(v).reshape(v.shape)[:12, 0]).all()


# ---------------------------------------------------------------- P12 integer maps
def test_slot_map_and_cache_image_exact():
    wl = wk.make_workload(wk.Config("t", "bf16", 3, 4, 2, 8, 32, 64, ("list", [37, 16, 1]), ("list", [3, 0, 9])),
                          seed=5, lm=False)
    table, nb = wl.block_table, wl.num_blocks
    used = set()
    for s in range(3):
        for t in range(int(wl.prompt_lens[s])):
            sl = oracle.slot(table, s, t)
            assert sl == int(table[s, t // 16]) * 16 + t % 16
            assert sl not in used
            used.add(sl)
    kp, vp = wl.prefix_pack(wl.k), wl.prefix_pack(wl.v)
    kc, vc = oracle.cache_image(kp, vp, wl.cu_prefix, table, nb, sentinel=0x7FC1)
    flat_k = kc.transpose(0, 2, 1, 3).reshape(nb * 16, 2, 8)
    flat_v = vc.transpose(0, 2, 1, 3).reshape(nb * 16, 2, 8)
    for s in range(3):
        for t in range(int(wl.prompt_lens[s])):
            sl = oracle.slot(table, s, t)
            assert (flat_k[sl] == kp[wl.cu_prefix[s] + t]).all()
            assert (flat_v[sl] == vp[wl.cu_prefix[s] + t]).all()
    untouched = np.ones(nb * 16, bool)
    untouched[list(used)] = False
    assert (flat_k[untouched] == 0x7FC1).all() and (flat_v[untouched] == 0x7FC1).all()
    assert untouched.sum() == nb * 16 - 54


# ---------------------------------------------------------------- P8 split == monolithic, P10
def _split_form(wl, table):
    """Independent split evaluation (numpy fp64): prefix rows from the prefix alone; suffix rows
    from [bf16 cache read back through the block table ; suffix K/V]."""
    cfg = wl.cfg
    g = cfg.num_q_heads // cfg.num_kv_heads
    scale = 1.0 / math.sqrt(cfg.head_dim)
    f = lambda a: wk.bf16_bits_to_f32(a).reshape(a.shape).astype(np.float64)
    qp, kp, vp = (wl.prefix_pack(t) for t in (wl.q, wl.k, wl.v))
    qs, ks, vs = (f(wl.suffix_pack(t)) for t in (wl.q, wl.k, wl.v))
    kc, vc = oracle.cache_image(kp, vp, wl.cu_prefix, table, wl.num_blocks)
    kc = f(kc).transpose(0, 2, 1, 3).reshape(-1, cfg.num_kv_heads, cfg.head_dim)
    vc = f(vc).transpose(0, 2, 1, 3).reshape(-1, cfg.num_kv_heads, cfg.head_dim)
    qp, kp, vp = f(qp), f(kp), f(vp)
    out = np.zeros((wl.n_tokens, cfg.num_q_heads, cfg.head_dim))

    def soft(qrow, keys, vals):
        s = keys @ qrow * scale
        p = np.exp(s - s.max())
        return (p[:, None] * vals).sum(axis=0) / p.sum()

    for s in range(cfg.batch):
        p, r = int(wl.prompt_lens[s]), int(wl.response_lens[s])
        a = int(wl.cu_full[s])
        slots = np.array([oracle.slot(table, s, t) for t in range(p)], np.int64)
        for h in range(cfg.num_q_heads):
            kvh = h // g
            for i in range(p):
                lo = int(wl.cu_prefix[s])
                out[a + i, h] = soft(qp[lo + i, h], kp[lo: lo + i + 1, kvh], vp[lo: lo + i + 1, kvh])
            for i in range(r):
                lo = int(wl.cu_suffix[s])
                keys = np.concatenate([kc[slots, kvh], ks[lo: lo + i + 1, kvh]])
                vals = np.concatenate([vc[slots, kvh], vs[lo: lo + i + 1, kvh]])
                out[a + p + i, h] = soft(qs[lo + i, h], keys, vals)
    return out


def test_split_scoring_equals_monolithic_and_block_shuffle_is_invisible():
    cfg = wk.Config("t", "bf16", 4, 4, 2, 8, 32, 64, ("list", [21, 0, 16, 5]), ("list", [4, 6, 0, 1]))
    wl = wk.make_workload(cfg, seed=7, lm=False)
    rows = oracle.all_rows(wl.cu_full, cfg.num_q_heads)
    mono, _ = oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, rows)
    mono = mono.reshape(wl.n_tokens, cfg.num_q_heads, cfg.head_dim)
    split = _split_form(wl, wl.block_table)
    np.testing.assert_allclose(split, mono, rtol=0, atol=1e-12)
    # another physical placement of the same logical blocks changes nothing
    other, _ = wk.make_block_table(wl.prompt_lens, seed=1234)
    assert not np.array_equal(other, wl.block_table)
    wl2 = wk.make_workload(cfg, seed=7, lm=False)
    wl2.block_table = other
    assert (_split_form(wl2, other) == split).all()


def test_prefix_logprobs_concatenated_with_suffix_logprobs_are_the_full_values():
    cfg = wk.Config("t", "bf16", 2, 2, 1, 8, 16, 50, ("list", [5, 3]), ("list", [2, 4]))
    wl = wk.make_workload(cfg, seed=9, attn=False)
    full, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    pre, _ = oracle.logprob_rows(wl.prefix_pack(wl.hidden), wl.w, wl.prefix_pack(wl.ids))
    suf, _ = oracle.logprob_rows(wl.suffix_pack(wl.hidden), wl.w, wl.suffix_pack(wl.ids))
    merged = np.empty_like(full)
    merged[wl.prefix_rows()] = pre
    merged[wl.suffix_rows()] = suf
    assert (merged == full).all()


# ---------------------------------------------------------------- P11 input statistics
def test_tiny_config_statistics_match_the_recipe():
    wl = wk.make_workload(wk.CONFIGS["C1"], seed=0)
    assert wl.n_prefix == 256 and wl.n_suffix == 32 and wl.q.dtype == np.float32
    assert abs(float(wl.w.std()) - 0.02) < 2e-4 and abs(float(wl.hidden.std()) - 1.0) < 2e-2
    assert wl.ids.min() >= 0 and wl.ids.max() < 4096
    lp, lse = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    expect = -(math.log(4096) + 0.5 * 256 * 0.02**2)  # E[lse] = ln V + var(z)/2 for Gaussian logits
    assert abs(lp.mean() - expect) < 0.08
    assert abs(lse.mean() + expect) < 0.02
    # determinism and thread-count independence of the generator
    wl_b = wk.make_workload(wk.CONFIGS["C1"], seed=0)
    assert (wl.q == wl_b.q).all() and (wl.w == wl_b.w).all() and (wl.ids == wl_b.ids).all()


def test_length_recipes():
    for name, lo_share, hi_share in [("C2", 0.94, 0.942), ("C3", 0.88, 0.96), ("C4", 0.984, 0.986), ("C5", 0.12, 0.20)]:
        cfg = wk.CONFIGS[name]
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([0, 7, 0])))
        p = wk.draw_lengths(cfg.prompt, cfg.batch, rng)
        r = wk.draw_lengths(cfg.response, cfg.batch, rng)
        share = p.sum() / (p.sum() + r.sum())
        assert lo_share <= share <= hi_share, (name, share)
    p = wk.draw_lengths(("lognormal", 6000, 0.5, 1024, 16384), 2000, np.random.default_rng(0))
    assert p.min() >= 1024 and p.max() <= 16384 and abs(np.median(p) - 6000) < 300


# ---------------------------------------------------------------- entropy (extension) pins
def test_entropy_closed_forms_bounds_and_torch():
    vocab, h = 64, 12
    hid = _rand((5, h), 200)
    # uniform distribution: ln V
    ent = oracle.entropy_rows(hid, np.zeros((vocab, h), np.float32))
    assert np.abs(ent - math.log(vocab)).max() < 1e-13
    # two classes with logits (a, 0): the binary entropy of sigmoid(a), typed out independently
    w2 = np.zeros((2, h), np.float32)
    w2[0, 0] = 1.0
    hid2 = np.zeros((4, h), np.float32)
    hid2[:, 0] = [0.0, 1.5, -3.0, 30.0]
    ent2 = oracle.entropy_rows(hid2, w2)
    for a, got in zip([0.0, 1.5, -3.0, 30.0], ent2):
        p1 = 1.0 / (1.0 + math.exp(-a))
        ref = -(p1 * math.log(p1) + (1 - p1) * math.log1p(-p1)) if p1 < 1.0 else 0.0
        assert abs(got - ref) < 1e-12
    # bounds, and the library routine in fp64
    w = _rand((vocab, h), 201, 0.7)
    ent3 = oracle.entropy_rows(hid, w)
    assert (ent3 > 0).all() and (ent3 < math.log(vocab)).all()
    logits = torch.from_numpy(hid).double() @ torch.from_numpy(w).double().T
    ref = torch.distributions.Categorical(logits=logits).entropy().numpy()
    np.testing.assert_allclose(ent3, ref, rtol=0, atol=1e-12)
    # consistency with the log-prob oracle: H = lse - E_p[z]
    _, lse = oracle.logprob_rows(hid, w, np.zeros(5, np.int32))
    z = logits.numpy()
    pr = np.exp(z - lse[:, None])
    np.testing.assert_allclose(ent3, lse - (pr * z).sum(axis=1), rtol=0, atol=1e-12)
    sub = oracle.entropy_rows(hid, w, rows=np.array([4, 1], np.int64))
    assert (sub == ent3[[4, 1]]).all()
