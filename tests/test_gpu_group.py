"""cfgzip_group_tokens (grouping of tokens with equal displacement signature on the GPU) against the CPU oracle's
grouping, bit for bit: class ids, representatives, class count and class lists. Cases: the toy grammars end to end
(signatures from Algorithm 1, grouped on the GPU, loaded as a partition and used by a decode step), degenerate
vocabularies, and a Llama-size vocabulary of synthetic signatures checked against numpy's unique-rows routine."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import offline
from synth import rng
from paper_2605_29986_b200 import binding as cz
from _gpu_util import Ctx, compare_step, dev, oracle_step, run_fused
from test_offline_host import library_signatures

pytestmark = pytest.mark.gpu


def gpu_group(sig, lens, lists=True):
    V, W = sig.shape
    d_sig, d_len = dev(np.ascontiguousarray(sig, dtype=np.int32)), dev(np.asarray(lens, dtype=np.int32))
    d_c = torch.full((V,), -7, dtype=torch.int32, device="cuda")
    d_r = torch.full((V,), -7, dtype=torch.int32, device="cuda")
    d_k = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    d_off = torch.full((V + 1,), -7, dtype=torch.int32, device="cuda") if lists else None
    d_tok = torch.full((V,), -7, dtype=torch.int32, device="cuda") if lists else None
    cz.cfgzip_group_tokens(d_sig, W, d_len, V, d_c, d_r, d_k, d_off, d_tok, torch.cuda.current_stream())
    K = int(d_k.cpu()[0])
    return (d_c.cpu().numpy(), d_r.cpu().numpy()[:K], K, None if not lists else d_off.cpu().numpy(),
            None if not lists else d_tok.cpu().numpy())


def check_against_oracle(sig, lens):
    want_c, want_r = offline.group_tokens([tuple(row) for row in sig], list(lens))
    c, r, K, off, tok = gpu_group(sig, lens)
    assert K == len(want_r) and c.tolist() == want_c and r.tolist() == want_r
    want_off, want_tok = oracle.build_csr(np.asarray(want_c, dtype=np.int32), K)
    assert np.array_equal(off[:K + 1], want_off) and np.all(off[K + 1:] == len(want_c)) and np.array_equal(tok, want_tok)
    c2, r2, K2, _, _ = gpu_group(sig, lens, lists=False)
    assert K2 == K and np.array_equal(c2, c) and np.array_equal(r2, r)
    return c, r, K


@pytest.mark.parametrize("name", ["figure3", "arithmetic", "json_like"])
def test_toy_grammar_from_signatures_to_a_decode_step(name):
    spec = synth.grammars.GRAMMARS[name]()
    tokens = synth.grammars.toy_vocabulary(spec, max_len=2, extra=60)
    _, sig, _, rc = library_signatures(spec, tokens)
    assert rc == cz.OK
    lens = [len(t) for t in tokens]
    c, r, K = check_against_oracle(sig, lens)
    # the partition the offline step produced is a valid input of the per-step path
    V = len(tokens)
    assert cz.cfgzip_check_partition(c, V, r, K) == cz.OK
    part = synth.Partition(V=V, K=K, c=c.astype(np.int32), r=r.astype(np.int32), sizes=np.bincount(c, minlength=K))
    cm = synth.class_mask_bernoulli(K, 5, 0.5, rng.stream_key(321))
    z = synth.logits_normal(5, V, 1.0, "f32", (322,))
    with Ctx([part]) as ctx:
        compare_step(run_fused(ctx, None, cm, z, V), oracle_step([part], None, cm, z, V), V)


def test_degenerate_vocabularies():
    check_against_oracle(np.array([[3, 1, 2, 0]], dtype=np.int32), [4])                         # one token
    check_against_oracle(np.zeros((70, 3), dtype=np.int32), list(range(70, 0, -1)))              # all equal: the last is shortest
    check_against_oracle(np.arange(200, dtype=np.int32).reshape(200, 1), [1] * 200)              # all different, one word
    same_len = np.array([[1, 7], [1, 8], [1, 7], [1, 7], [1, 8]], dtype=np.int32)
    c, r, K = check_against_oracle(same_len, [2, 2, 2, 2, 2])
    assert r.tolist() == [0, 1]                                                                   # ties: the lowest id


def test_rows_that_share_a_first_slot_are_still_told_apart():
    # 5000 tokens in 40 classes, many rows differing in the last word only: whatever the hash does with them, rows
    # that differ must land in different classes and equal rows in one
    base = (rng.u64(rng.stream_key(5), 40 * 6) % np.uint64(5)).astype(np.int32).reshape(40, 6)
    base[:, 5] = np.arange(40)
    which = (rng.u64(rng.stream_key(6), 5000) % np.uint64(40)).astype(np.int64)
    lens = (1 + rng.u64(rng.stream_key(7), 5000) % np.uint64(9)).astype(np.int32)
    check_against_oracle(base[which], lens)


def test_llama_size_vocabulary_of_synthetic_signatures():
    V, K, W = 128256, 2048, 8
    part = synth.zipf_partition(V, K, 1.1, seed=3)
    rows = (rng.u64(rng.stream_key(8), K * W) % np.uint64(7)).astype(np.int32).reshape(K, W)
    rows[:, 0] = W - 1
    rows[:, 1] = np.arange(K) // 7                 # many classes share most of their words
    rows[:, 2] = np.arange(K) % 7
    sig = rows[part.c]
    lens = (1 + rng.u64(rng.stream_key(9), V) % np.uint64(12)).astype(np.int32)
    c, r, Kg, off, tok = gpu_group(sig, lens)
    # numpy's unique rows give the classes; renumber them in the order of their lowest token id
    _, first, inverse = np.unique(sig, axis=0, return_index=True, return_inverse=True)
    order = np.argsort(first)
    rank = np.empty_like(order)
    rank[order] = np.arange(len(order))
    want_c = rank[inverse.reshape(-1)]
    assert Kg == K and np.array_equal(c, want_c)
    key = lens.astype(np.int64) * V + np.arange(V)
    want_r = np.full(K, np.iinfo(np.int64).max)
    np.minimum.at(want_r, want_c, key)
    assert np.array_equal(r, want_r % V)
    want_off, want_tok = oracle.build_csr(want_c.astype(np.int32), K)
    assert np.array_equal(off[:K + 1], want_off) and np.array_equal(tok, want_tok)
    # and a sample of it through the oracle's own grouping
    sub = np.sort(rng.permutation(rng.stream_key(10), V)[:1500])
    check_against_oracle(sig[sub], lens[sub])
