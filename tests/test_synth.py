"""The seeded input generators: exactness of the truncated Zipf sampler,
determinism, and the shapes of the five workloads (scaled down)."""
import numpy as np

from paper_1909_04823_b200 import synth


def test_zipf_truncated_matches_exact_pmf():
    rng = np.random.default_rng(0)
    for s, n in ((1.1, 50), (1.05, 1000), (1.2, 7)):
        N = 400_000
        x = synth.zipf_truncated(rng, s, n, N)
        assert x.min() >= 1 and x.max() <= n
        pmf = np.arange(1, n + 1, dtype=np.float64) ** -s
        pmf /= pmf.sum()
        cnt = np.bincount(x, minlength=n + 1)[1:]
        top = min(n, 20)
        z = (cnt[:top] - N * pmf[:top]) / np.sqrt(N * pmf[:top] * (1 - pmf[:top]))
        assert np.abs(z).max() < 5.0
        # tail mass beyond the top ranks
        if n > top:
            zt = (cnt[top:].sum() - N * pmf[top:].sum()) / np.sqrt(N * pmf[top:].sum())
            assert abs(zt) < 5.0


def test_fmix64_distinct_and_deterministic():
    a = synth.fmix64(np.arange(100000, dtype=np.uint64))
    assert np.unique(a).size == a.size
    assert np.array_equal(a, synth.fmix64(np.arange(100000, dtype=np.uint64)))


def test_workload_shapes_scaled():
    for i in range(1, 6):
        w = synth.config(i)
        w = w.scaled(batch=64, vocab=min(w.vocab, 5000) if w.vocab else 0,
                     prepopulate=1000 if w.prepopulate else 0)
        s1, s2 = synth.Stream(w), synth.Stream(w)
        b1, b2 = s1.next_batch(), s2.next_batch()
        assert np.array_equal(b1.ids, b2.ids) and np.array_equal(b1.offsets, b2.offsets)
        assert b1.offsets.shape == (64 * w.fields + 1,) and b1.offsets[0] == 0
        assert b1.offsets[-1] == b1.nnz and np.all(np.diff(b1.offsets) >= 0)
        lens = np.diff(b1.offsets)
        if w.len_law == "onehot":
            assert np.all(lens == 1)
        if i == 1:
            assert lens.min() >= 1 and lens.max() <= 4
        if i == 5:
            assert lens.max() <= 100 and 15 < lens.mean() < 25
        if i == 4:
            n0 = 1000
            assert s1.n_seen > n0 and abs((s1.n_seen - n0) / b1.nnz - w.p_new) < 0.03
            b3 = s1.next_batch()
            assert not np.array_equal(b3.ids[:50], b1.ids[:50])
        if i == 3:
            # bucketised fields use at most 64 ids each
            f_of = np.repeat(np.tile(np.arange(w.fields), 64), lens)
            for f in range(w.bucket_fields):
                assert np.unique(b1.ids[f_of == f]).size <= 64


def test_prepopulation_batch_layout():
    ids = synth.fmix64(np.arange(10, dtype=np.uint64))
    b = synth.prepopulation_batch(ids, 4)
    assert b.batch == 3 and b.offsets.shape == (13,) and b.offsets[-1] == 10
    assert list(np.diff(b.offsets)) == [1] * 10 + [0, 0]
