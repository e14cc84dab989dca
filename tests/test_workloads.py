"""The seeded input generators: determinism, documented shapes, slice/chunk consistency."""
import torch

from paper_2502_04677_b200 import workloads as W


def test_mixer_matches_published_splitmix64_vector():
    # first output of SplitMix64 seeded with 0 (published test vector of the generator)
    assert W.mix64_int(0) == 0xE220A8397B1DCDAF
    x = torch.tensor([0, 1, 2, 2**40 + 12345, -5], dtype=torch.int64)
    for a, b in zip(x.tolist(), W.mix64(x).tolist()):
        assert (b & ((1 << 64) - 1)) == W.mix64_int(a & ((1 << 64) - 1))


def test_tiny_shape_and_determinism():
    w = W.tiny()
    assert w.queries.n == 1000 and w.prefill.n == 2000 and w.vocab == 32000 and tuple(w.ks) == (2,)
    tok, off = w.queries.materialize()
    tok2, _ = W.tiny().queries.materialize()
    assert torch.equal(tok, tok2)
    lens = off[1:] - off[:-1]
    assert int(lens.min()) >= 512 + 64 and int(lens.max()) <= 512 + 256
    assert int(tok.min()) >= 0 and int(tok.max()) < 32000
    # exactly 8 distinct 512-token prefixes over queries and cached prompts together
    ttok, toff = w.prefill.materialize()
    heads = {tuple(tok[o:o + 512].tolist()) for o in off[:-1].tolist()} | \
            {tuple(ttok[o:o + 512].tolist()) for o in toff[:-1].tolist()}
    assert len(heads) == 8
    assert bool((w.arrivals[1:] >= w.arrivals[:-1]).all()) and w.start_tick == int(w.arrivals.max())


def test_slices_and_chunks_are_consistent():
    w = W.adversarial(scale=1 / 2048)
    tok, off = w.queries.materialize()
    a, _ = w.queries.materialize(chunk_tokens=5000)
    assert torch.equal(tok, a)
    b, _ = w.queries.materialize(lo=3, hi=11)
    assert torch.equal(b, tok[off[3]:off[11]])
    sub = w.queries.select(torch.tensor([5, 2, 9]))
    c, co = sub.materialize()
    assert torch.equal(c[co[1]:co[2]], tok[off[2]:off[3]])


def test_adversarial_queries_mismatch_one_token_past_the_trunk():
    w = W.adversarial(scale=1 / 2048)
    tok, off = w.queries.materialize()
    cut = w.queries.seg_end[0]
    key = w.queries.seg_key[0]
    for i in range(w.queries.n):
        cont = int(W._lsr(W.mix64(key[i:i + 1] + cut[i:i + 1]), 33) % w.vocab)
        assert int(tok[off[i] + cut[i]]) != cont


def test_configs_have_documented_sizes():
    m = W.medium()
    assert m.queries.n == 32768 and m.prefill.n == 100000 and tuple(m.ks) == (1, 2, 4, 8)
    h = W.hierarchical()
    assert h.queries.n == 65536 and h.prefill.n == 1_000_000
    s = W.streaming()
    assert s.budget_tokens == 50_000_000 and s.prefill.n == 0 and abs(s.queries.n - 120000) == 0
    a = W.adversarial()
    assert a.queries.n == 262144 and a.prefill.n == 2_000_000
    assert 2.0e9 < a.queries.total_tokens() < 2.4e9


def test_prefix_ratio_queue_shape():
    w = W.prefix_ratio(1000, 5000)
    assert w.queries.n == 2000 and w.prefill.n == 0 and w.budget_tokens == 0
    tok, off = w.queries.materialize()
    assert bool(((off[1:] - off[:-1]) == 6000).all())
    heads = {}
    for i, o in enumerate(off[:-1].tolist()):
        heads.setdefault(tuple(tok[o:o + 8].tolist()), []).append(i)
    assert len(heads) == 500 and all(len(v) == 4 for v in heads.values())     # every user prefix exactly 4 times
    # shuffled: the four replicas of a prefix are not adjacent in general
    assert any(max(v) - min(v) > 3 for v in heads.values())
    assert bool((w.arrivals[1:] >= w.arrivals[:-1]).all())
