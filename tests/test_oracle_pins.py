"""Pins for the CPU oracle: it is checked against things other than itself.

Closed forms, algebraic invariants, the corollary of the paper's Theorem 1 (a token and
the representative of its class always share a mask bit), a library log-softmax in
float64 on the case where the path reduces to a textbook one, a hand-worked example and
per-bit brute force on tiny shapes whose V and K are not multiples of 32.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import synth
from synth import rng

NEG_INF_F32 = np.uint32(0xFF800000)
NEG_INF_BF16 = np.uint16(0xFF80)


def _popcount_rows(words):
    return np.unpackbits(np.ascontiguousarray(words).view(np.uint8), axis=-1).sum(axis=-1)


def _rand_mask(K, B, p, *ids):
    return synth.class_mask_bernoulli(K, B, p, rng.stream_key(991, *ids))


SHAPES = [(1, 1), (31, 2), (32, 31), (33, 32), (63, 33), (64, 5), (65, 64), (1000, 37), (4099, 130)]


# ---------------------------------------------------------------- expand

def test_hand_worked_example():
    # six tokens, three classes; classes 0 and 2 allowed
    c = np.array([0, 1, 0, 2, 1, 2], dtype=np.int32)
    r = np.array([0, 1, 3], dtype=np.int32)
    cm = np.array([[0b101]], dtype=np.uint32)
    vm = oracle.expand_mask(c, 3, cm)
    assert vm.tolist() == [[0b101101]]  # tokens 0, 2, 3, 5
    z = np.array([[1.0, 5.0, 2.0, 0.0, 9.0, 2.0]], dtype=np.float32)
    oracle.mask_logits(z, 6, vm)
    assert z[0, [0, 2, 3, 5]].tolist() == [1.0, 2.0, 0.0, 2.0]
    assert np.all(np.isneginf(z[0, [1, 4]]))
    am, lse, lpa, full = oracle.logsoftmax_argmax(z, 6, vm, want_full=True)
    assert am.tolist() == [2]  # 2.0 appears at tokens 2 and 5: the lower id wins
    want_lse = math.log(math.e + 2 * math.e ** 2 + 1.0)
    assert abs(lse[0] - want_lse) < 1e-12
    assert abs(lpa[0] - (2.0 - want_lse)) < 1e-12
    assert abs(full[0, 3] - (0.0 - want_lse)) < 1e-12 and np.isneginf(full[0, 1])
    assert oracle.map_tokens(c, r, am).tolist() == [0]


@pytest.mark.parametrize("V,K", SHAPES)
def test_expand_brute_force_per_bit(V, K):
    K = min(K, V)
    part = synth.zipf_partition(V, K, 1.1, seed=V + K)
    cm = _rand_mask(K, 3, 0.4, V, K)
    vm = oracle.expand_mask(part.c, K, cm)
    assert vm.shape == (3, (V + 31) // 32)
    for b in range(3):
        for i in range(V):
            k = int(part.c[i])
            want = (int(cm[b, k // 32]) >> (k % 32)) & 1
            got = (int(vm[b, i // 32]) >> (i % 32)) & 1
            assert got == want, (b, i)
        for i in range(V, 32 * vm.shape[1]):  # tail bits of the last word are zero
            assert (int(vm[b, i // 32]) >> (i % 32)) & 1 == 0


@pytest.mark.parametrize("V,K", [(1000, 37), (32000, 256), (128256, 2048)])
def test_expand_popcount_equals_allowed_class_sizes(V, K):
    part = synth.zipf_partition(V, K, 1.1, seed=3)
    sizes = np.bincount(part.c, minlength=K)
    cm = _rand_mask(K, 4, 0.3, V)
    vm = oracle.expand_mask(part.c, K, cm)
    allowed = synth.unpack_bits(cm, K)
    assert _popcount_rows(vm).tolist() == (allowed * sizes[None, :]).sum(axis=1).tolist()


@pytest.mark.parametrize("V,K", SHAPES)
def test_expand_all_ones_all_zeros_and_ignored_tail_bits(V, K):
    K = min(K, V)
    part = synth.zipf_partition(V, K, 1.1, seed=1)
    KW = (K + 31) // 32
    ones = np.full((1, KW), 0xFFFFFFFF, dtype=np.uint32)  # includes garbage bits >= K
    vm = oracle.expand_mask(part.c, K, ones)
    assert synth.unpack_bits(vm, 32 * vm.shape[1])[0].tolist() == [i < V for i in range(32 * vm.shape[1])]
    assert not oracle.expand_mask(part.c, K, np.zeros((1, KW), dtype=np.uint32)).any()
    cm = _rand_mask(K, 2, 0.5, V, K, 7)
    dirty = cm.copy()
    if K % 32:
        dirty[:, -1] |= np.uint32((0xFFFFFFFF << (K % 32)) & 0xFFFFFFFF)
    assert np.array_equal(oracle.expand_mask(part.c, K, cm), oracle.expand_mask(part.c, K, dirty))


@pytest.mark.parametrize("V", [1, 31, 32, 33, 100, 1024])
def test_expand_identity_partition_copies_the_class_mask(V):
    part = synth.identity_partition(V)
    cm = _rand_mask(V, 3, 0.5, V)
    assert np.array_equal(oracle.expand_mask(part.c, V, cm), cm)


def test_expand_single_class_is_all_or_nothing():
    c = np.zeros(77, dtype=np.int32)
    on = oracle.expand_mask(c, 1, np.array([[1]], dtype=np.uint32))
    off = oracle.expand_mask(c, 1, np.array([[0]], dtype=np.uint32))
    assert _popcount_rows(on).tolist() == [77] and _popcount_rows(off).tolist() == [0]


def test_expand_is_a_boolean_homomorphism():
    V, K = 5003, 211
    part = synth.zipf_partition(V, K, 1.1, seed=5)
    a, b = _rand_mask(K, 2, 0.5, 1), _rand_mask(K, 2, 0.3, 2)
    ea, eb = oracle.expand_mask(part.c, K, a), oracle.expand_mask(part.c, K, b)
    assert np.array_equal(oracle.expand_mask(part.c, K, a | b), ea | eb)
    assert np.array_equal(oracle.expand_mask(part.c, K, a & b), ea & eb)
    valid = synth.pack_bits(np.ones((1, V), dtype=bool))
    assert np.array_equal(oracle.expand_mask(part.c, K, ~a), ~ea & valid)


def test_expand_invariant_under_class_relabelling():
    V, K = 3001, 97
    part = synth.zipf_partition(V, K, 1.1, seed=6)
    perm = rng.permutation(rng.stream_key(5, 5), K)  # new id of class k is perm[k]
    bits = synth.unpack_bits(_rand_mask(K, 3, 0.4, 9), K)
    bits2 = np.zeros_like(bits)
    bits2[:, perm] = bits
    c2 = perm[part.c].astype(np.int32)
    assert np.array_equal(oracle.expand_mask(part.c, K, synth.pack_bits(bits)),
                          oracle.expand_mask(c2, K, synth.pack_bits(bits2)))


@pytest.mark.parametrize("maker", ["zipf", "heavy"])
def test_token_and_its_representative_share_a_bit(maker):
    # corollary of Theorem 1: feeding the engine r_{c_t} instead of t changes nothing
    V, K = 20000, 300
    part = (synth.zipf_partition(V, K, 1.1, seed=8) if maker == "zipf"
            else synth.heavy_tail_partition(V, K, 0.6, 1.3, seed=8))
    vm = oracle.expand_mask(part.c, K, _rand_mask(K, 4, 0.2, 3))
    bits = synth.unpack_bits(vm, V)
    reps = part.r[part.c]
    assert np.array_equal(bits, bits[:, reps])


@pytest.mark.parametrize("V,K", SHAPES + [(32000, 256)])
def test_dense_and_class_side_expansion_agree(V, K):
    K = min(K, V)
    part = synth.zipf_partition(V, K, 1.1, seed=2)
    off, tok = oracle.build_csr(part.c, K)
    assert off[0] == 0 and off[-1] == V
    assert np.array_equal(np.diff(off), np.bincount(part.c, minlength=K))
    assert sorted(tok.tolist()) == list(range(V))
    for k in range(K):
        seg = tok[off[k]:off[k + 1]]
        assert np.all(part.c[seg] == k) and np.all(np.diff(seg) > 0)
    cm = _rand_mask(K, 3, 0.3, V, 4)
    assert np.array_equal(oracle.expand_mask(part.c, K, cm), oracle.expand_mask_csr(off, tok, V, K, cm))


# ---------------------------------------------------------------- mask_logits

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mask_logits_identities(dtype):
    V, stride, B = 1003, 1010, 3
    z0 = synth.logits_normal(B, stride, 1.0, dtype, (1, 2, 3))
    ones = synth.pack_bits(np.ones((B, V), dtype=bool))
    z = z0.copy()
    oracle.mask_logits(z, V, ones)
    assert np.array_equal(z.view(np.uint8), z0.view(np.uint8))  # all allowed: bit-identical
    z = z0.copy()
    oracle.mask_logits(z, V, np.zeros_like(ones))
    ninf = NEG_INF_F32 if dtype == "f32" else NEG_INF_BF16
    bits = z.view(np.uint32 if dtype == "f32" else np.uint16)
    assert np.all(bits[:, :V] == ninf)
    assert np.array_equal(bits[:, V:], z0.view(bits.dtype)[:, V:])  # beyond V untouched
    vm = synth.pack_bits(rng.uniform(rng.stream_key(4), B * V).reshape(B, V) < 0.3)
    z = z0.copy()
    oracle.mask_logits(z, V, vm)
    once = z.copy()
    oracle.mask_logits(z, V, vm)
    assert np.array_equal(z.view(np.uint8), once.view(np.uint8))  # idempotent
    bits = once.view(np.uint32 if dtype == "f32" else np.uint16)
    keep = synth.unpack_bits(vm, V)
    assert np.array_equal(bits[:, :V][keep], z0.view(bits.dtype)[:, :V][keep])
    assert np.all(bits[:, :V][~keep] == ninf)
    assert ((bits[:, :V] == ninf).sum(axis=1) == V - _popcount_rows(vm)).all()


# ---------------------------------------------------------------- log-softmax / argmax

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_logsoftmax_reduces_to_library_routine_when_everything_is_allowed(dtype):
    V, B = 4001, 5
    z = synth.logits_normal(B, V, 2.0, dtype, (7, 7))
    ones = synth.pack_bits(np.ones((B, V), dtype=bool))
    am, lse, lpa, full = oracle.logsoftmax_argmax(z, V, ones, want_full=True)
    if dtype == "bf16":
        zt = torch.from_numpy(z.view(np.int16)).view(torch.bfloat16).to(torch.float64)
    else:
        zt = torch.from_numpy(z).to(torch.float64)
    ref = torch.log_softmax(zt, dim=-1).numpy()
    assert np.allclose(full, ref, rtol=0, atol=1e-10)
    assert np.allclose(lse, torch.logsumexp(zt, dim=-1).numpy(), rtol=0, atol=1e-10)
    assert am.tolist() == [int(np.flatnonzero(row == row.max())[0]) for row in zt.numpy()]
    assert np.allclose(lpa, ref[np.arange(B), am], rtol=0, atol=1e-10)


def test_logsoftmax_masked_equals_library_routine_on_the_allowed_subset():
    V, B = 3000, 4
    z = synth.logits_normal(B, V, 1.0, "f32", (8, 1))
    keep = rng.uniform(rng.stream_key(8, 2), B * V).reshape(B, V) < 0.2
    vm = synth.pack_bits(keep)
    oracle.mask_logits(z, V, vm)
    am, lse, lpa, full = oracle.logsoftmax_argmax(z, V, vm, want_full=True)
    for b in range(B):
        idx = np.flatnonzero(keep[b])
        sub = torch.from_numpy(z[b, idx]).to(torch.float64)
        ref = torch.log_softmax(sub, dim=-1).numpy()
        assert np.allclose(full[b, idx], ref, rtol=0, atol=1e-10)
        assert np.all(np.isneginf(full[b, ~keep[b]]))
        assert am[b] == idx[int(np.argmax(sub.numpy()))]
        assert abs(np.exp(full[b, idx]).sum() - 1.0) < 1e-9


def test_logsoftmax_closed_forms():
    V = 777
    for n, a in [(1, 3.5), (7, -2.0), (777, 0.25)]:
        z = np.full((1, V), a, dtype=np.float32)
        keep = np.zeros((1, V), dtype=bool)
        keep[0, rng.permutation(rng.stream_key(n), V)[:n]] = True
        vm = synth.pack_bits(keep)
        oracle.mask_logits(z, V, vm)
        am, lse, lpa, _ = oracle.logsoftmax_argmax(z, V, vm)
        assert abs(lse[0] - (a + math.log(n))) < 1e-12
        assert abs(lpa[0] + math.log(n)) < 1e-12
        assert am[0] == np.flatnonzero(keep[0])[0]  # constant row: lowest allowed id


def test_logsoftmax_shift_invariance_and_sign():
    V, B = 2000, 3
    z = synth.logits_normal(B, V, 1.0, "f32", (9, 1))
    vm = synth.pack_bits(rng.uniform(rng.stream_key(9, 2), B * V).reshape(B, V) < 0.5)
    z2 = (z + np.float32(4.0)).astype(np.float32)
    oracle.mask_logits(z, V, vm)
    oracle.mask_logits(z2, V, vm)
    a1, l1, p1, f1 = oracle.logsoftmax_argmax(z, V, vm, want_full=True)
    a2, l2, p2, f2 = oracle.logsoftmax_argmax(z2, V, vm, want_full=True)
    assert np.array_equal(a1, a2)
    assert np.allclose(l2 - l1, 4.0, atol=1e-5)  # float32 rounding of the shifted inputs
    fin = np.isfinite(f1)
    assert np.allclose(f1[fin], f2[fin], atol=1e-5)
    assert np.all(p1 <= 0.0)


def test_argmax_planted_spikes_and_ties():
    V, K = 5000, 64
    part = synth.zipf_partition(V, K, 1.1, seed=11)
    bits = np.zeros((1, K), dtype=bool)
    bits[0, :20] = True
    cm = synth.pack_bits(bits)
    allowed = np.flatnonzero(bits[0][part.c])
    masked = np.flatnonzero(~bits[0][part.c])
    z0 = synth.logits_normal(1, V, 1.0, "f32", (12,))

    def run(z):
        return oracle.decode_step([part], None, cm, z.copy())

    z = z0.copy(); z[0, allowed[37]] = 50.0
    assert run(z)["argmax"][0] == allowed[37]
    z = z0.copy(); z[0, allowed[90]] = 50.0; z[0, allowed[12]] = 50.0
    assert run(z)["argmax"][0] == allowed[12]  # equal maxima: lower id
    z = z0.copy(); z[0, masked[5]] = 99.0; z[0, allowed[41]] = 50.0
    out = run(z)
    assert out["argmax"][0] == allowed[41]  # a spike at a disallowed token is never returned
    assert synth.unpack_bits(out["vocab_mask"], V)[0, out["argmax"][0]]
    z = np.full((1, V), -3.0, dtype=np.float32); z[0, allowed[7]] = 0.0; z[0, allowed[3]] = -0.0
    assert run(z)["argmax"][0] == allowed[3]  # -0.0 == +0.0: a tie, lower id wins
    brute = max(allowed, key=lambda i: (z0[0, i], -i))
    assert run(z0)["argmax"][0] == brute


def test_degenerate_rows():
    V, K = 100, 4
    part = synth.zipf_partition(V, K, 1.1, seed=1)
    z = synth.logits_normal(2, V, 1.0, "f32", (13,))
    cm = np.array([[0], [0b10]], dtype=np.uint32)
    z[1, part.c == 1] = -np.inf  # every allowed logit of row 1 is -inf
    out = oracle.decode_step([part], None, cm, z, want_full=True)
    assert out["argmax"][0] == -1 and out["rep"][0] == -1
    assert np.isneginf(out["lse"][0]) and np.isneginf(out["logp_argmax"][0])
    assert np.all(np.isneginf(z[0])) and not out["vocab_mask"][0].any()
    assert out["argmax"][1] == np.flatnonzero(part.c == 1)[0]
    assert out["rep"][1] == part.r[1]
    assert np.isneginf(out["lse"][1]) and np.all(np.isneginf(out["logp_full"][1]))


# ---------------------------------------------------------------- map_tokens / whole step

def test_map_tokens_algebra():
    V, K = 9000, 150
    part = synth.zipf_partition(V, K, 1.1, seed=14)
    assert np.array_equal(part.c[part.r], np.arange(K))  # c[r_k] = k
    toks = np.arange(V, dtype=np.int32)
    m = oracle.map_tokens(part.c, part.r, toks)
    assert np.array_equal(oracle.map_tokens(part.c, part.r, m), m)  # idempotent
    assert np.array_equal(part.c[m], part.c)  # stays inside the class
    assert np.all(m <= toks)  # representative is the lowest id of the class
    assert oracle.map_tokens(part.c, part.r, np.array([-1, V, V + 5], dtype=np.int32)).tolist() == [-1, -1, -1]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_decode_step_is_the_composition_of_its_steps_and_handles_row_partitions(dtype):
    V, K, B = 2500, 70, 6
    parts = [synth.zipf_partition(V, K, 1.1, seed=s) for s in range(3)]
    row_part = np.array([0, 1, 2, 2, 1, 0], dtype=np.int32)
    cm = _rand_mask(K, B, 0.3, 15)
    z0 = synth.logits_normal(B, V, 2.0, dtype, (15,))
    z = z0.copy()
    out = oracle.decode_step(parts, row_part, cm, z, want_full=True, threads=3)
    for b in range(B):
        p = parts[row_part[b]]
        vm = oracle.expand_mask(p.c, K, cm[b:b + 1])
        zb = z0[b:b + 1].copy()
        oracle.mask_logits(zb, V, vm)
        am, lse, lpa, full = oracle.logsoftmax_argmax(zb, V, vm, want_full=True)
        assert np.array_equal(out["vocab_mask"][b:b + 1], vm)
        assert np.array_equal(z[b:b + 1].view(np.uint8), zb.view(np.uint8))
        assert out["argmax"][b] == am[0] and out["lse"][b] == lse[0] and out["logp_argmax"][b] == lpa[0]
        assert np.array_equal(out["logp_full"][b], full[0])
        assert out["rep"][b] == p.r[p.c[am[0]]]


def test_bf16_ties_go_to_the_lowest_id():
    # bf16 logits over thousands of allowed tokens tie at the maximum routinely
    V = 128256
    z = synth.logits_normal(1, V, 2.0, "bf16", (16,))
    ones = synth.pack_bits(np.ones((1, V), dtype=bool))
    am, _, _, _ = oracle.logsoftmax_argmax(z, V, ones)
    f = rng.bf16_bits_to_f32(z[0])
    assert am[0] == np.flatnonzero(f == f.max())[0]


# ---------------------------------------------------------------- sampling (inverse CDF at a temperature)

def _full_mask(V):
    return synth.pack_bits(np.ones((1, V), dtype=bool))


def test_sample_hand_worked_example():
    # allowed tokens 0, 2, 3, 5 with weights 1 : 2 : 3 : 4 (logits = their logs), tokens 1 and 4 masked
    w = np.array([1.0, 7.0, 2.0, 3.0, 9.0, 4.0])
    z = np.log(w).astype(np.float32)[None, :]
    vm = synth.pack_bits(np.array([[1, 0, 1, 1, 0, 1]], dtype=bool))
    oracle.mask_logits(z, 6, vm)
    # cumulative probabilities over the allowed tokens: 0.1, 0.3, 0.6, 1.0
    for u, want in [(0.0, 0), (0.05, 0), (0.15, 2), (0.29, 2), (0.31, 3), (0.59, 3), (0.61, 5), (0.999999, 5)]:
        tok, lse, lpt, cdf = oracle.sample(z.copy(), 6, vm, 1.0, [u], want_cdf=True)
        assert tok.tolist() == [want], (u, tok)
        assert abs(lse[0] - math.log(10.0)) < 1e-6
        assert abs(lpt[0] - math.log(w[want] / 10.0)) < 1e-6
        assert np.allclose(cdf[0], [0.1, 0.1, 0.3, 0.6, 0.6, 1.0], atol=1e-7)
    # temperature 1/2 squares the weights: 1 : 4 : 9 : 16 -> cumulative 1/30, 5/30, 14/30, 1
    for u, want in [(0.03, 0), (0.04, 2), (0.16, 2), (0.17, 3), (0.46, 3), (0.47, 5)]:
        tok, lse, lpt, _ = oracle.sample(z.copy(), 6, vm, 2.0, [u])
        assert tok.tolist() == [want], (u, tok)
        assert abs(lse[0] - math.log(30.0)) < 1e-5
        assert abs(lpt[0] - math.log(w[want] ** 2 / 30.0)) < 1e-5


def test_sample_equal_logits_closed_form():
    # n equal allowed logits: token = the floor(u*n)-th allowed one, lse = a/T + log n, logp = -log n
    V, n = 1000, 37
    allowed = np.sort(rng.permutation(rng.stream_key(5, 1), V)[:n])
    bits = np.zeros((1, V), dtype=bool)
    bits[0, allowed] = True
    vm = synth.pack_bits(bits)
    z = np.full((1, V), 1.5, dtype=np.float32)
    oracle.mask_logits(z, V, vm)
    for u in [0.0, 0.013, 0.25, 0.5, 0.77, 0.99]:
        tok, lse, lpt, _ = oracle.sample(z.copy(), V, vm, 4.0, [u])
        assert tok[0] == allowed[int(u * n)]
        assert abs(lse[0] - (1.5 * 4.0 + math.log(n))) < 1e-12 and abs(lpt[0] + math.log(n)) < 1e-12


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sample_matches_library_cumsum_search(dtype):
    # away from its boundaries the inverse CDF is numpy's searchsorted on the cumulative softmax of the allowed subset
    V, K, B = 3000, 40, 6
    part = synth.zipf_partition(V, K, 1.1, seed=9)
    cm = _rand_mask(K, B, 0.3, 77)
    z = synth.logits_normal(B, V, 2.0, dtype, (4, 4))
    vm = oracle.expand_mask(part.c, K, cm)
    oracle.mask_logits(z, V, vm)
    zf = rng.bf16_bits_to_f32(z.reshape(-1)).reshape(B, V) if dtype == "bf16" else z
    for inv_t in (1.0, 5.0):
        for trial in range(5):
            u = rng.uniform(rng.stream_key(8, trial), B)
            tok, lse, lpt, _ = oracle.sample(z.copy(), V, vm, inv_t, u)
            for b in range(B):
                idx = np.flatnonzero(synth.unpack_bits(vm[b:b + 1], V)[0])
                p = torch.softmax(torch.from_numpy(zf[b, idx].astype(np.float64)) * inv_t, dim=0).numpy()
                cdf = np.cumsum(p)
                j = int(np.searchsorted(cdf, u[b], side="right"))
                if min(abs(cdf - u[b])) < 1e-9:
                    continue  # on a boundary: rounding order decides
                assert tok[b] == idx[j]
                assert abs(lpt[b] - math.log(p[j])) < 1e-9
                want_lse = torch.logsumexp(torch.from_numpy(zf[b, idx].astype(np.float64)) * inv_t, dim=0).item()
                assert abs(lse[b] - want_lse) < 1e-9


def test_sample_stratified_uniforms_reproduce_the_distribution():
    # N evenly spaced u hit token i between N*p_i - 1 and N*p_i + 1 times: a property of any inverse CDF,
    # so a wrong sum, order or normalisation anywhere shows up as a wrong count
    V, N = 50, 20000
    z = (rng.normal_f32(rng.stream_key(6, 6), V, 1.5))[None, :].astype(np.float32)
    bits = np.ones((1, V), dtype=bool)
    bits[0, ::7] = False
    vm = synth.pack_bits(bits)
    oracle.mask_logits(z, V, vm)
    inv_t = 1.0 / 0.7
    p = np.where(bits[0], np.exp((z[0].astype(np.float64) - z[0][bits[0]].max()) * inv_t), 0.0)
    p /= p.sum()
    us = (np.arange(N) + 0.5) / N
    zz = np.repeat(z, N, axis=0)
    vv = np.repeat(vm, N, axis=0)
    tok, _, _, _ = oracle.sample(zz, V, vv, inv_t, us)
    counts = np.bincount(tok, minlength=V)
    assert np.all(np.abs(counts - N * p) <= 1.0 + 1e-6)
    assert counts[::7].sum() == 0  # a masked token is never drawn
    assert np.all(np.diff(tok) >= 0)  # monotone in u


def test_sample_temperature_identities():
    V = 400
    z = rng.normal_f32(rng.stream_key(6, 7), V, 1.0)[None, :].astype(np.float32)
    vm = _full_mask(V)
    u = rng.uniform(rng.stream_key(6, 8), 64)
    zz, vv = np.repeat(z, 64, axis=0), np.repeat(vm, 64, axis=0)
    # halving the temperature = doubling the logits (exact in float32)
    t_a, lse_a, lp_a, _ = oracle.sample(zz.copy(), V, vv, 2.0, u)
    t_b, lse_b, lp_b, _ = oracle.sample((2.0 * zz).astype(np.float32), V, vv, 1.0, u)
    assert np.array_equal(t_a, t_b) and np.allclose(lse_a, lse_b, atol=1e-12) and np.allclose(lp_a, lp_b, atol=1e-12)
    # T = 1: lse is the greedy path's lse, and a cold distribution collapses onto the argmax
    am, lse_g, _, _ = oracle.logsoftmax_argmax(zz.copy(), V, vv)
    _, lse_1, _, _ = oracle.sample(zz.copy(), V, vv, 1.0, u)
    assert np.allclose(lse_1, lse_g, atol=1e-12)
    t_cold, _, lp_cold, _ = oracle.sample(zz.copy(), V, vv, 1000.0, np.minimum(u, 0.999))
    assert np.array_equal(t_cold, am) and np.all(lp_cold > -1e-3)
    # adding a constant to the row moves lse by constant/T and nothing else (logits on a 1/64 grid: the shift is exact)
    zq = (np.round(zz * 64.0) / 64.0).astype(np.float32)
    t_q, lse_q, lp_q, _ = oracle.sample(zq.copy(), V, vv, 2.0, u)
    t_s, lse_s, lp_s, _ = oracle.sample((zq + np.float32(4.0)).astype(np.float32), V, vv, 2.0, u)
    assert np.array_equal(t_s, t_q) and np.allclose(lse_s, lse_q + 8.0, atol=1e-12) and np.allclose(lp_s, lp_q, atol=1e-12)


def test_sample_degenerate_rows_and_last_token():
    V = 70
    z = np.zeros((3, V), dtype=np.float32)
    bits = np.zeros((3, V), dtype=bool)
    bits[1, [5, 40]] = True
    bits[2, [3, 66]] = True
    z[1, [5, 40]] = -np.inf          # allowed, but both -inf
    vm = synth.pack_bits(bits)
    oracle.mask_logits(z, V, vm)
    tok, lse, lpt, cdf = oracle.sample(z, V, vm, 1.0, [0.5, 0.5, 0.999999999], want_cdf=True)
    assert tok.tolist() == [-1, 5, 66]
    assert np.isneginf(lse[:2]).all() and np.isneginf(lpt[:2]).all()
    assert abs(lse[2] - math.log(2.0)) < 1e-12 and cdf[2, 66] == 1.0 and cdf[2, 3] == 0.5


def test_sample_step_is_the_composition_of_its_steps():
    w = synth.make_workload(4, B=16, V=5000, K=300)
    cm, z, u = w.class_masks(0), w.logits(0), w.uniforms(0)
    assert u.dtype == np.float32 and np.all((u >= 0) & (u < 1))
    z1 = z.copy()
    out = oracle.sample_step(w.partitions, w.row_part, cm, z1, 5.0, u, threads=2)
    for b in range(w.B):
        p = w.partition_of_row(b)
        vm = oracle.expand_mask(p.c, p.K, cm[b:b + 1])
        zb = z[b:b + 1].copy()
        oracle.mask_logits(zb, w.V, vm)
        tok, lse, lpt, _ = oracle.sample(zb, w.V, vm, 5.0, u[b:b + 1])
        assert np.array_equal(vm[0], out["vocab_mask"][b]) and np.array_equal(zb[0], z1[b])
        assert tok[0] == out["token"][b] and lse[0] == out["lse"][b] and lpt[0] == out["logp_token"][b]
        assert oracle.map_tokens(p.c, p.r, tok)[0] == out["rep"][b]
        t = int(tok[0])
        assert (int(vm[0, t // 32]) >> (t % 32)) & 1 == 1


# ------------------------------------------------------------------ several masks per logits row

def test_multi_mask_hand_worked_example():
    # six tokens in three classes (0, 1, 2, 0, 1, 2), logits 1..6; mask {0} allows tokens 0 and 3, mask {1, 2} the rest
    part = synth.Partition(V=6, K=3, c=np.array([0, 1, 2, 0, 1, 2], dtype=np.int32), r=np.array([0, 1, 2], dtype=np.int32),
                           sizes=np.array([2, 2, 2]))
    z = np.array([[1.0, 2.0, 3.0, 4.0, 5.0, 6.0]], dtype=np.float32)
    cms = np.array([[0b001], [0b110]], dtype=np.uint32)
    out = oracle.multi_mask_step(part, cms, 2, z)
    assert out["argmax"].tolist() == [3, 5] and out["rep"].tolist() == [0, 2]
    assert out["vocab_mask"][:, 0].tolist() == [0b001001, 0b110110]
    assert abs(out["lse"][0] - math.log(math.exp(1.0) + math.exp(4.0))) < 1e-12
    assert abs(out["lse"][1] - math.log(math.exp(2.0) + math.exp(3.0) + math.exp(5.0) + math.exp(6.0))) < 1e-12
    assert abs(out["logp_argmax"][0] - (4.0 - out["lse"][0])) < 1e-12
    assert z.tolist() == [[1.0, 2.0, 3.0, 4.0, 5.0, 6.0]]  # the logits are left alone


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_multi_mask_is_one_step_per_mask_and_order_free(dtype):
    V, K, B, M = 3001, 77, 5, 4
    part = synth.zipf_partition(V, K, 1.1, seed=3)
    z = synth.logits_normal(B, V, 2.0, dtype, (21,))
    cms = synth.class_mask_bernoulli(K, B * M, 0.3, rng.stream_key(22))
    cms[6] = 0                                     # one (row, mask) with nothing allowed
    z0 = z.copy()
    out = oracle.multi_mask_step(part, cms, M, z)
    assert np.array_equal(z.view(np.uint8), z0.view(np.uint8))
    # one mask per row is the plain step
    one = oracle.multi_mask_step(part, cms[::M], 1, z)
    plain = oracle.decode_step([part], None, cms[::M], z.copy())
    for key in ("vocab_mask", "argmax", "rep", "lse", "logp_argmax"):
        assert np.array_equal(one[key], plain[key]), key
        assert np.array_equal(out[key][::M], plain[key]), key
    # the masks of a row do not see one another: reversing their order reverses the results
    rev = cms.reshape(B, M, -1)[:, ::-1].reshape(B * M, -1)
    out_rev = oracle.multi_mask_step(part, rev, M, z)
    for key in ("vocab_mask", "argmax", "rep", "lse", "logp_argmax"):
        got = out_rev[key].reshape((B, M) + out_rev[key].shape[1:])[:, ::-1].reshape(out[key].shape)
        assert np.array_equal(got, out[key]), key
    assert out["argmax"][6] == -1 and out["rep"][6] == -1 and np.isneginf(out["lse"][6])


def test_multi_mask_disjoint_masks_add_up():
    # masks A and B allow disjoint class sets, C = A | B: the allowed tokens split, so the normalisers add and the
    # greedy choice under C is the better of the two choices (the lower token id on a tie)
    V, K, B = 4000, 64, 6
    part = synth.zipf_partition(V, K, 1.1, seed=4)
    z = synth.logits_normal(B, V, 2.0, "bf16", (23,))      # bf16: ties at the maximum do occur
    a = synth.class_mask_bernoulli(K, B, 0.4, rng.stream_key(24))
    b = synth.class_mask_bernoulli(K, B, 0.4, rng.stream_key(25)) & ~a
    cms = np.stack([a, b, a | b], axis=1).reshape(B * 3, -1)
    out = oracle.multi_mask_step(part, cms, 3, z)
    zf = rng.bf16_bits_to_f32(z.reshape(-1)).reshape(z.shape).astype(np.float64)
    for row in range(B):
        ia, ib, ic = 3 * row, 3 * row + 1, 3 * row + 2
        assert np.array_equal(out["vocab_mask"][ic], out["vocab_mask"][ia] | out["vocab_mask"][ib])
        assert not np.any(out["vocab_mask"][ia] & out["vocab_mask"][ib])
        assert abs(math.exp(out["lse"][ic]) - math.exp(out["lse"][ia]) - math.exp(out["lse"][ib])) <= 1e-9 * math.exp(out["lse"][ic])
        ta, tb = int(out["argmax"][ia]), int(out["argmax"][ib])
        best = max((zf[row, ta], -ta), (zf[row, tb], -tb))
        assert out["argmax"][ic] == -best[1]


# ------------------------------------------------------------------ top-k / top-p sampling

def _weights_row(ws):
    """One row whose tempered weights at T = 1 are ws (logits log w), all allowed."""
    z = np.log(np.asarray(ws, dtype=np.float64)).astype(np.float32)[None, :]
    return z, _full_mask(len(ws))


def test_filtered_sampling_hand_worked():
    # weights 1 : 2 : 3 : 4 on tokens 0..3
    z, vm = _weights_row([1, 2, 3, 4])
    def run(k, p, u):
        return oracle.sample_filtered(z.copy(), 4, vm, 1.0, k, p, [u], want_kept=True)
    o = run(2, 1.0, 0.4)                                  # top-2 keeps tokens 3 and 2 (weights 4 and 3): CDF 3/7, 1
    assert o["kept"][0].tolist() == [0, 0, 1, 1] and o["n_kept"][0] == 2 and o["token"][0] == 2
    assert abs(o["lse"][0] - math.log(7.0)) < 1e-6 and abs(o["logp_token"][0] - math.log(3.0 / 7.0)) < 1e-6
    assert run(2, 1.0, 0.5)["token"][0] == 3
    o = run(0, 0.5, 0.0)                                  # top-p 0.5 of 10: 4 < 5 <= 4 + 3 keeps tokens 3 and 2
    assert o["kept"][0].tolist() == [0, 0, 1, 1] and abs(o["p_margin"][0] - 0.1) < 1e-6
    assert run(0, 0.39, 0.0)["kept"][0].tolist() == [0, 0, 0, 1]     # 3.9 <= 4: the top token alone
    assert run(0, 0.71, 0.0)["kept"][0].tolist() == [0, 1, 1, 1]     # 7 < 7.1 <= 9
    o = run(3, 0.5, 0.99)                                 # top-3 first (weights 4, 3, 2 = 9), then half of 9: 4 < 4.5 <= 7
    assert o["kept"][0].tolist() == [0, 0, 1, 1] and o["token"][0] == 3


def test_filtered_sampling_ties_keep_the_lowest_ids():
    z, vm = _weights_row([5, 2, 5, 5, 1, 5])             # four equal maxima at tokens 0, 2, 3, 5
    o = oracle.sample_filtered(z.copy(), 6, vm, 1.0, 2, 1.0, [0.0], want_kept=True)
    assert o["kept"][0].tolist() == [1, 0, 1, 0, 0, 0]
    o = oracle.sample_filtered(z.copy(), 6, vm, 1.0, 0, 0.6, [0.0], want_kept=True)     # 0.6 * 23 = 13.8: three maxima
    assert o["kept"][0].tolist() == [1, 0, 1, 1, 0, 0]


def test_filtered_sampling_reduces_to_the_plain_cases():
    V = 700
    z = rng.normal_f32(rng.stream_key(9, 1), 6 * V, 2.0).reshape(6, V)
    bits = rng.uniform(rng.stream_key(9, 2), 6 * V).reshape(6, V) < 0.4
    vm = synth.pack_bits(bits)
    oracle.mask_logits(z, V, vm)
    u = rng.uniform(rng.stream_key(9, 3), 6)
    plain = oracle.sample(z.copy(), V, vm, 5.0, u)
    allowed = bits.sum(axis=1)
    for k, p in ((0, 1.0), (int(allowed.max()), 1.0), (V + 5, 1.5)):                      # no filter at all
        o = oracle.sample_filtered(z.copy(), V, vm, 5.0, k, p, u)
        assert np.array_equal(o["token"], plain[0]) and np.allclose(o["lse"], plain[1], atol=1e-12)
        assert np.allclose(o["logp_token"], plain[2], atol=1e-12) and np.all(o["n_kept"] == allowed)
    am, _, _, _ = oracle.logsoftmax_argmax(z.copy(), V, vm)
    for uu in (0.0, 0.5, 0.999999):                                                        # top-1 is the greedy choice
        o = oracle.sample_filtered(z.copy(), V, vm, 5.0, 1, 1.0, [uu] * 6)
        assert np.array_equal(o["token"], am) and np.allclose(o["logp_token"], 0.0, atol=1e-12)
        o = oracle.sample_filtered(z.copy(), V, vm, 5.0, 0, 1e-9, [uu] * 6)                # a tiny top-p too
        assert np.array_equal(o["token"], am)


def test_filtered_sampling_keeps_a_top_set_of_the_right_size_and_weight():
    V, B = 3000, 8
    z = rng.normal_f32(rng.stream_key(9, 4), B * V, 2.0).reshape(B, V)
    bits = rng.uniform(rng.stream_key(9, 5), B * V).reshape(B, V) < 0.5
    vm = synth.pack_bits(bits)
    oracle.mask_logits(z, V, vm)
    u = rng.uniform(rng.stream_key(9, 6), B)
    for k, p, inv_t in ((50, 1.0, 1.0), (0, 0.9, 1.0), (200, 0.5, 2.0), (7, 0.999, 5.0)):
        o = oracle.sample_filtered(z.copy(), V, vm, inv_t, k, p, u, want_kept=True)
        for b in range(B):
            kept = o["kept"][b].astype(bool)
            assert not np.any(kept & ~bits[b]) and kept[o["token"][b]]
            assert z[b][kept].min() >= z[b][bits[b] & ~kept].max()           # nothing dropped beats anything kept
            w = np.exp((z[b].astype(np.float64) - z[b][bits[b]].max()) * inv_t)
            if p >= 1.0:
                assert kept.sum() == min(k, bits[b].sum())
            else:
                top = np.sort(w[bits[b]])[::-1][: (k or V)]
                target = p * top.sum()
                assert w[kept].sum() >= target * (1 - 1e-12)                  # reaches the target ...
                assert w[kept].sum() - w[kept].min() < target * (1 + 1e-12)  # ... and would not without its last token
            assert abs(o["lse"][b] - (float(z[b][bits[b]].max()) * inv_t + math.log(w[kept].sum()))) < 1e-9


def test_filtered_sampling_degenerate_rows():
    V = 40
    z = np.zeros((2, V), dtype=np.float32)
    bits = np.zeros((2, V), dtype=bool)
    bits[1, [7, 30]] = True
    z[1, [7, 30]] = -np.inf
    vm = synth.pack_bits(bits)
    oracle.mask_logits(z, V, vm)
    o = oracle.sample_filtered(z, V, vm, 1.0, 3, 0.5, [0.3, 0.3])
    assert o["token"].tolist() == [-1, 7] and np.isneginf(o["lse"]).all() and np.isneginf(o["logp_token"]).all()
