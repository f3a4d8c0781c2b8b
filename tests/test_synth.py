"""The synthetic-input recipes: shapes follow the paper's Table 1, streams are reproducible."""
import os

import numpy as np
import pytest
import torch

import synth
from synth import rng

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_vocab_classes.txt")


def _table1():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows.append((f[0], int(f[1]), [float(x) for x in f[2:]]))
    return rows


def test_splitmix64_matches_its_published_sequence():
    # first outputs of SplitMix64 seeded with 0 and with 1234567 (reference vectors of the algorithm)
    assert [int(v) for v in rng.u64(np.uint64(0), 3)] == [
        0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert [int(v) for v in rng.u64(np.uint64(1234567), 2)] == [6457827717110365317, 3203168211198807973]


def test_streams_are_counter_based_and_distinct():
    k = rng.stream_key(1, 2, 3)
    assert np.array_equal(rng.u64(k, 10, offset=5), rng.u64(k, 15)[5:])
    assert rng.stream_key(1, 2, 3) != rng.stream_key(1, 3, 2)
    x = rng.normal_f32(k, 200001, 2.0)
    assert abs(x.mean()) < 0.02 and abs(x.std() - 2.0) < 0.02 and np.isfinite(x).all()


def test_bf16_rounding_is_nearest_even():
    x = rng.normal_f32(rng.stream_key(5), 100000, 3.0)
    ours = rng.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    assert np.array_equal(rng.bf16_bits_to_f32(ours),
                          torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).float().numpy())


def test_configs_match_the_papers_vocabularies():
    vocab = {v for _, v, _ in _table1()}
    ks = [k for _, _, row in _table1() for k in row]
    for cfg in (2, 3, 5):
        assert synth.CONFIGS[cfg]["V"] in vocab
    assert min(ks) * 0.9 < synth.CONFIGS[1]["K"] < max(ks) * 1.5
    # compression ratios quoted by the paper: about 40:1 to about 800:1
    lo = min(v / max(row) for _, v, row in _table1())
    hi = max(v / min(row) for _, v, row in _table1())
    assert 38 < lo < 45 and 750 < hi < 850
    for cfg in (2, 3, 5):
        ratio = synth.CONFIGS[cfg]["V"] / synth.CONFIGS[cfg]["K"]
        assert 30 < ratio < 850
    # c and r together stay under a megabyte for 100k-200k vocabularies (int32 entries)
    for _, v, row in _table1():
        assert 4 * (v + max(row)) < 1_000_000


@pytest.mark.parametrize("V,K,s", [(32000, 256, 1.1), (128256, 2048, 1.1), (1000, 1000, 1.1), (50, 7, 1.1)])
def test_zipf_partition_is_a_valid_partition(V, K, s):
    p = synth.zipf_partition(V, K, s, seed=0, config=9)
    assert p.c.dtype == np.int32 and p.c.shape == (V,) and p.r.shape == (K,)
    sizes = np.bincount(p.c, minlength=K)
    assert sizes.min() >= 1 and sizes.sum() == V and np.array_equal(sizes, p.sizes)
    assert np.array_equal(p.c[p.r], np.arange(K))
    first = np.full(K, V)
    np.minimum.at(first, p.c, np.arange(V))
    assert np.array_equal(first, p.r)  # representative = lowest id in the class
    q = synth.zipf_partition(V, K, s, seed=0, config=9)
    assert np.array_equal(p.c, q.c)
    if K > 1 and V > K:
        assert not np.array_equal(p.c, synth.zipf_partition(V, K, s, seed=1, config=9).c)


def test_zipf_largest_class_share():
    p = synth.zipf_partition(128256, 2048, 1.1, seed=0)
    assert 0.12 < p.sizes.max() / 128256 < 0.25
    # members of a class are scattered, not contiguous
    big = np.flatnonzero(p.c == np.argmax(p.sizes))
    assert big.max() - big.min() > 100000


def test_heavy_tail_partition():
    V, K = 256000, 16384
    p = synth.heavy_tail_partition(V, K, 0.6, 1.3, seed=3)
    assert p.sizes[0] == 153600 and p.sizes.min() >= 1 and p.sizes.sum() == V
    assert np.array_equal(p.c[p.r], np.arange(K))


def test_pack_unpack_roundtrip_and_bit_order():
    bits = np.zeros((1, 70), dtype=bool)
    bits[0, [0, 33, 69]] = True
    w = synth.pack_bits(bits)
    assert w.tolist() == [[1, 2, 32]]
    assert np.array_equal(synth.unpack_bits(w, 70), bits)


def test_class_mask_recipes():
    m = synth.class_mask_bernoulli(2048, 64, 0.1, rng.stream_key(1))
    assert m.shape == (64, 64)
    dens = synth.unpack_bits(m, 2048).mean()
    assert 0.09 < dens < 0.11
    m = synth.class_mask_n_classes(512, 200, 1, 5, rng.stream_key(2))
    n = synth.unpack_bits(m, 512).sum(axis=1)
    assert n.min() >= 1 and n.max() <= 5 and len(set(n.tolist())) == 5
    m = synth.class_mask_bernoulli(100, 4, np.array([0.0, 1.0, 0.5, 0.5]), rng.stream_key(3))
    b = synth.unpack_bits(m, 100)
    assert b[0].sum() == 0 and b[1].sum() == 100
    assert (m[:, -1] >> np.uint32(4)).max() == 0  # bits >= K are zero


def test_workloads_shapes():
    w = synth.make_workload(4, B=16, V=4096, K=512)
    assert len(w.partitions) == 8 and w.row_part.tolist() == [b % 8 for b in range(16)]
    assert w.class_masks(0).shape == (16, 16) and w.logits(0).dtype == np.uint16
    assert not np.array_equal(w.class_masks(0), w.class_masks(1))
    w = synth.make_workload(3, B=8, V=5000, K=128)
    z = w.logits(2)
    assert z.dtype == np.float32 and z.shape == (8, 5000)
    assert ((z > 5.5).sum(axis=1) >= 40).all()  # the +8 spikes
    w = synth.make_workload(5, B=8, V=5000, K=128)
    assert synth.unpack_bits(w.class_masks(0), 128).sum(axis=1).max() <= 5
