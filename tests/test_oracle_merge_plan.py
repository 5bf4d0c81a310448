"""Pins for the oracle's merge (row scatter / gather) and planning rule, and for the seeded
workload recipes.  Merge and plan are integer / bit-exact work: each has one correct result."""
import numpy as np
import pytest

import oracle
from paper_2607_03229_b200 import workloads as W


def test_merge_rows_by_hand():
    enc = np.arange(3 * 4, dtype=np.uint16).reshape(3, 4) + 100
    emb = np.arange(6 * 4, dtype=np.uint16).reshape(6, 4)
    out = oracle.merge_tokens(enc, emb, [4, 0, 3])
    expect = emb.copy()
    expect[4], expect[0], expect[3] = enc[0], enc[1], enc[2]
    assert np.array_equal(out, expect)
    assert np.array_equal(emb, np.arange(24, dtype=np.uint16).reshape(6, 4))  # input untouched


def test_merge_properties():
    w = W.tiny(shuffled_positions=True)
    enc, emb, pos = w.merge_source(), w.llm_embeds(), w.positions
    out = oracle.merge_tokens(enc, emb, pos)
    assert np.array_equal(out[pos], enc)                     # gather(out, pos) == enc
    rest = np.setdiff1d(np.arange(w.n_llm_tokens), pos)
    assert np.array_equal(out[rest], emb[rest])              # rows not in pos unchanged
    assert np.array_equal(oracle.merge_tokens(enc[:0], emb, pos[:0]), emb)   # nothing to merge
    ident = np.arange(229, dtype=np.int32)
    assert np.array_equal(oracle.merge_tokens(enc, emb[:229], ident), enc)   # identity -> plain copy
    assert np.array_equal(oracle.merge_tokens_bwd(out, pos), enc)            # reverse seam reads them back
    with pytest.raises(AssertionError):
        oracle.merge_tokens(enc[:1], emb, [512])


def _recount(counts, tile):
    """Brute force: walk every token, record which (segment, tile) it falls in."""
    seen = {}
    tok = 0
    for s, n in enumerate(counts):
        for r in range(n):
            seen.setdefault((s, r // tile), []).append(tok)
            tok += 1
    return seen


@pytest.mark.parametrize("trained", [False, True])
def test_plan_invariants_and_recount(trained):
    rng = np.random.default_rng(0)
    for trial in range(40):
        n_seg = int(rng.integers(0, 9))
        counts = [int(x) for x in rng.integers(0, 700, size=n_seg)]
        if trial % 5 == 0 and n_seg:
            counts[0] = 0
        cu, T, mx, fwd, bwd = oracle.seg_plan(counts, 256, 128, trained)
        assert cu[0] == 0 and len(cu) == n_seg + 1 and T == sum(counts) == cu[-1]
        assert all(cu[i + 1] - cu[i] == counts[i] for i in range(n_seg))
        assert mx == (max(counts) if counts else 0)
        if not trained:
            assert bwd == []
        for items, tile in ((fwd, 256), (bwd, 128) if trained else (fwd, 256)):
            seen = _recount(counts, tile)
            assert len(items) == len(seen)
            assert sorted((it[0], it[1]) for it in items) == sorted(seen)
            assert sum(it[3] for it in items) == T
            for seg, t, r0, rl, k0, kl in items:
                toks = seen[(seg, t)]
                assert r0 == toks[0] and rl == len(toks) and k0 == cu[seg] and kl == counts[seg]
                assert 1 <= rl <= tile and cu[seg] <= r0 and r0 + rl <= cu[seg + 1]
            kls = [it[5] for it in items]
            assert kls == sorted(kls, reverse=True)          # longest segments first
            # ties keep the original segment order, tiles ascend inside a segment
            keyed = [(-it[5], it[0], it[1]) for it in items]
            assert keyed == sorted(keyed)


def test_plan_worked_example():
    """Four images of 16, 49, 64 and 100 patches with 64-row tiles, written out by hand."""
    cu, T, mx, fwd, bwd = oracle.seg_plan([16, 49, 64, 100], 64, 64, True)
    assert cu == [0, 16, 65, 129, 229] and T == 229 and mx == 100
    assert fwd == [(3, 0, 129, 64, 129, 100), (3, 1, 193, 36, 129, 100), (2, 0, 65, 64, 65, 64),
                   (1, 0, 16, 49, 16, 49), (0, 0, 0, 16, 0, 16)]
    assert bwd == fwd


def test_workload_recipes_are_reproducible_and_in_range():
    a, b = W.vit_l(), W.vit_l()
    assert a.patch_counts == b.patch_counts and len(a.patch_counts) == 32
    assert all(256 <= n <= 4096 for n in a.patch_counts)
    q3 = W.qwen2vl()
    assert q3.total_tokens == 65536 and all(n <= 16384 for n in q3.patch_counts)
    assert all(n >= 64 for n in q3.patch_counts[:-1])
    v4 = W.video_tail()
    assert sorted(v4.patch_counts)[-4:] == [16384] * 4 and len(v4.patch_counts) == 204
    assert all(64 <= n <= 256 for n in sorted(v4.patch_counts)[:200])
    for f, tok in zip(W.MIX_FRACTIONS, (0, 6552, 16384, 32768, 49152)):
        m = W.modality_mix(f)
        assert m.total_tokens == tok and m.positions.size == tok
        assert np.unique(m.positions).size == tok
        if tok:
            assert m.positions.min() >= 0 and m.positions.max() < 65536
            # every image is one contiguous run inside a single 8192-token sequence
            cu = m.cu_seqlens
            for s in range(len(m.patch_counts)):
                p = m.positions[cu[s]:cu[s + 1]]
                assert np.array_equal(p, np.arange(p[0], p[0] + p.size)) and p[0] // 8192 == p[-1] // 8192
    t = W.tiny()
    assert t.total_tokens == 229 and np.unique(t.positions).size == 229 and t.positions.max() < 512
    ts = W.tiny(shuffled_positions=True)
    assert np.unique(ts.positions).size == 229 and not np.array_equal(np.sort(ts.positions), ts.positions)


def test_normal_generator_statistics_and_determinism():
    x = W.bf16_bits_to_f64(W.normal_bf16(123, 1, (1 << 18,)))
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert abs((x ** 3).mean()) < 0.03 and abs((x ** 4).mean() - 3.0) < 0.08
    assert np.array_equal(W.normal_bf16(123, 1, (1000,)), W.normal_bf16(123, 1, (1 << 18,))[:1000])
    assert not np.array_equal(W.normal_bf16(123, 1, (1000,)), W.normal_bf16(123, 2, (1000,)))
