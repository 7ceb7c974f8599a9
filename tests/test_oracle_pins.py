"""Pins for the CPU oracle: each check ties it to something other than itself
(closed forms, invariants, a library routine, a differently written brute
force, hand-worked fixtures), so that a dropped term, a wrong sign or index, or
a swapped operand in the oracle fails at least one of them."""
import math
import os

import numpy as np
import pytest

from oracle import attention as oa
from oracle import plan as op
from paper_2605_23296_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rand_bits(rng, shape):
    return bf(rng.standard_normal(shape, dtype=np.float32))


def brute_force_block(q, k, v, scale):
    """Dense mask-matrix softmax attention for ONE block, written independently
    of the oracle (matrix form, einsum, explicit -inf mask)."""
    L, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    qf, kf, vf = (oa.bf16_bits_to_f64(t) for t in (q, k, v))
    krep = np.repeat(kf, G, axis=1)           # kv head g serves q heads gG..gG+G-1
    vrep = np.repeat(vf, G, axis=1)
    s = np.einsum("ihc,jhc->hij", qf, krep) * scale
    mask = np.triu(np.ones((L, L), dtype=bool), k=1)
    s = np.where(mask[None], -np.inf, s)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return np.einsum("hij,jhc->ihc", p, vrep)


# ----------------------------------------------------------------------------
# closed forms
# ----------------------------------------------------------------------------

def test_two_key_closed_form():
    # d=2, q=(2,0); k0=(0,5), k1=(1,-3); scale 1 -> scores 0, 2
    q = bf([[[2.0, 0.0]], [[2.0, 0.0]]])
    k = bf([[[0.0, 5.0]], [[1.0, -3.0]]])
    v = bf([[[1.0, -2.0]], [[3.0, 4.0]]])
    out = oa.prefill(q, k, v, [0, 2], scale=1.0, threads=1)
    np.testing.assert_array_equal(out[0, 0], [1.0, -2.0])
    w1 = math.exp(2.0) / (1.0 + math.exp(2.0))
    np.testing.assert_allclose(out[1, 0], [1 + 2 * w1, -2 + 6 * w1], rtol=1e-14)
    # the scale multiplies the scores: scale 0.5 -> scores 0, 1
    out = oa.prefill(q, k, v, [0, 2], scale=0.5, threads=1)
    w1 = math.e / (1.0 + math.e)
    np.testing.assert_allclose(out[1, 0], [1 + 2 * w1, -2 + 6 * w1], rtol=1e-14)


def test_zero_keys_give_running_mean_of_values():
    rng = np.random.default_rng(0)
    L, Hq, Hkv, d = 37, 4, 2, 8
    q = rand_bits(rng, (L, Hq, d))
    k = np.zeros((L, Hkv, d), dtype=np.uint16)
    v = rand_bits(rng, (L, Hkv, d))
    out = oa.prefill(q, k, v, [0, L], scale=0.3)
    vf = oa.bf16_bits_to_f64(v)
    mean = np.cumsum(vf, axis=0) / np.arange(1, L + 1)[:, None, None]
    np.testing.assert_allclose(out, np.repeat(mean, Hq // Hkv, axis=1), rtol=1e-13, atol=1e-15)


def test_gqa_head_map_is_contiguous_groups():
    # K = 0 -> uniform weights; V of kv head g is the constant g -> out[h] = h div G
    L, Hq, Hkv, d = 5, 6, 3, 4
    q = rand_bits(np.random.default_rng(1), (L, Hq, d))
    k = np.zeros((L, Hkv, d), dtype=np.uint16)
    v = bf(np.broadcast_to(np.arange(Hkv, dtype=np.float32)[None, :, None], (L, Hkv, d)))
    out = oa.prefill(q, k, v, [0, L], scale=1.0)
    for h in range(Hq):
        np.testing.assert_allclose(out[:, h, :], h // 2, atol=1e-15)


def test_softmax_rows_sum_to_one_and_order():
    rng = np.random.default_rng(2)
    n, Hq, Hkv, d = 50, 4, 2, 16
    q = rand_bits(rng, (Hq, d))
    k = rand_bits(rng, (n, Hkv, d))
    v = rand_bits(rng, (n, Hkv, d))
    out, p = oa.attend_token(q, k, v, scale=0.25, return_weights=True)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=1e-14)
    assert (p > 0).all()
    # weights are monotone in the score and reproduce the output
    qf, kf, vf = (oa.bf16_bits_to_f64(t) for t in (q, k, v))
    for h in range(Hq):
        s = kf[:, h // 2, :] @ qf[h]
        assert (np.argsort(s) == np.argsort(p[h])).all()
        np.testing.assert_allclose(p[h] @ vf[:, h // 2, :], out[h], rtol=1e-12, atol=1e-14)
        # ratio of two weights is exp(scale * score difference)
        np.testing.assert_allclose(p[h, 3] / p[h, 7], math.exp(0.25 * (s[3] - s[7])), rtol=1e-12)


def test_single_visible_key_returns_its_value_exactly():
    w = wl.tiny(seed=11).materialise(with_decode=False)
    cu = np.concatenate([[0], np.cumsum(w.block_lens)])
    out = oa.prefill(w.q, w.k, w.v, cu, w.scale, rows=cu[:-1])
    vf = oa.bf16_bits_to_f64(w.v)
    for r, start in enumerate(cu[:-1]):
        np.testing.assert_array_equal(out[r], np.repeat(vf[start], 4, axis=0))
    # a block of length 1
    one = oa.prefill(w.q[:1], w.k[:1], w.v[:1], [0, 1], w.scale)
    np.testing.assert_array_equal(one[0], np.repeat(vf[0], 4, axis=0))


# ----------------------------------------------------------------------------
# invariants
# ----------------------------------------------------------------------------

def test_block_diagonal_batch_equals_each_block_alone_bitwise():
    w = wl.tiny(seed=3).materialise(with_decode=False)
    cu = np.concatenate([[0], np.cumsum(w.block_lens)])
    full = oa.prefill(w.q, w.k, w.v, cu, w.scale)
    for b in range(w.num_blocks):
        s, e = cu[b], cu[b + 1]
        alone = oa.prefill(w.q[s:e], w.k[s:e], w.v[s:e], [0, e - s], w.scale, threads=1)
        np.testing.assert_array_equal(full[s:e], alone)


def test_row_subset_equals_full_rows_bitwise():
    w = wl.tiny(seed=4).materialise(with_decode=False)
    cu = np.concatenate([[0], np.cumsum(w.block_lens)])
    full = oa.prefill(w.q, w.k, w.v, cu, w.scale)
    rows = np.array([0, 95, 96, 97, 255, 256, 479, 480, 767])
    sub = oa.prefill(w.q, w.k, w.v, cu, w.scale, rows=rows, threads=3)
    np.testing.assert_array_equal(sub, full[rows])


def test_causal_mask_future_tokens_do_not_matter():
    rng = np.random.default_rng(5)
    L, Hq, Hkv, d = 40, 2, 1, 8
    q, k, v = rand_bits(rng, (L, Hq, d)), rand_bits(rng, (L, Hkv, d)), rand_bits(rng, (L, Hkv, d))
    base = oa.prefill(q, k, v, [0, L], 0.35)
    i = 17
    k2, v2 = k.copy(), v.copy()
    k2[i + 1:] = rand_bits(rng, (L - i - 1, Hkv, d))
    v2[i + 1:] = rand_bits(rng, (L - i - 1, Hkv, d))
    pert = oa.prefill(q, k2, v2, [0, L], 0.35)
    np.testing.assert_array_equal(base[: i + 1], pert[: i + 1])
    assert np.abs(base[i + 1:] - pert[i + 1:]).max() > 1e-3      # later rows do see them
    # ... and the row's own key IS visible (j <= i, not j < i)
    k3 = k.copy()
    k3[i] = rand_bits(rng, (Hkv, d))
    assert np.abs(oa.prefill(q, k3, v, [0, L], 0.35)[i] - base[i]).max() > 1e-6


def test_shift_of_all_keys_leaves_output_unchanged():
    rng = np.random.default_rng(6)
    L, Hq, Hkv, d = 24, 4, 2, 8
    # multiples of 1/8 below 4 stay exact in bf16 after adding a multiple of 1/8 below 4
    q = bf(rng.integers(-16, 17, (L, Hq, d)) / 8.0)
    kq = rng.integers(-16, 17, (L, Hkv, d)) / 8.0
    v = rand_bits(rng, (L, Hkv, d))
    shift = rng.integers(-16, 17, (1, Hkv, d)) / 8.0
    a = oa.prefill(q, bf(kq), v, [0, L], 0.5)
    b = oa.prefill(q, bf(kq + shift), v, [0, L], 0.5)
    assert np.array_equal(oa.bf16_bits_to_f64(bf(kq + shift)), kq + shift)
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-12)


def test_gqa_equals_mha_with_repeated_kv_heads():
    rng = np.random.default_rng(7)
    L, Hq, Hkv, d = 33, 8, 2, 16
    q, k, v = rand_bits(rng, (L, Hq, d)), rand_bits(rng, (L, Hkv, d)), rand_bits(rng, (L, Hkv, d))
    gqa = oa.prefill(q, k, v, [0, L], 0.25)
    mha = oa.prefill(q, np.repeat(k, 4, axis=1), np.repeat(v, 4, axis=1), [0, L], 0.25)
    np.testing.assert_array_equal(gqa, mha)


def test_outlier_key_limit():
    # a key aligned with q and scaled up takes all the weight -> output -> its value
    rng = np.random.default_rng(8)
    n, d = 64, 32
    q = rand_bits(rng, (1, d))
    k = rand_bits(rng, (n, 1, d))
    v = rand_bits(rng, (n, 1, d))
    qf = oa.bf16_bits_to_f64(q)[0]
    prev = None
    for factor in (0.25, 0.5, 1.0, 2.0, 16.0):
        k2 = k.copy()
        k2[20, 0] = bf(qf * factor)
        out = oa.attend_token(q, k2, v, scale=1.0 / math.sqrt(d))
        err = np.abs(out[0] - oa.bf16_bits_to_f64(v)[20, 0]).max()
        if prev is not None:
            assert err < prev
        prev = err
    assert prev < 1e-12


# ----------------------------------------------------------------------------
# against a library routine and a brute force
# ----------------------------------------------------------------------------

def test_single_block_mha_matches_torch_sdpa_fp64():
    import torch
    import torch.nn.functional as F
    rng = np.random.default_rng(9)
    L, H, d = 70, 3, 16
    q, k, v = rand_bits(rng, (L, H, d)), rand_bits(rng, (L, H, d)), rand_bits(rng, (L, H, d))
    ours = oa.prefill(q, k, v, [0, L], 1.0 / math.sqrt(d))
    tq, tk, tv = (torch.from_numpy(oa.bf16_bits_to_f64(t)).permute(1, 0, 2)[None] for t in (q, k, v))
    ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(ours, ref, rtol=1e-11, atol=1e-13)


def test_tiny_config_against_dense_brute_force():
    w = wl.tiny(seed=0).materialise(with_decode=False)
    cu = np.concatenate([[0], np.cumsum(w.block_lens)])
    out = oa.prefill(w.q, w.k, w.v, cu, w.scale)
    for b in range(w.num_blocks):
        s, e = cu[b], cu[b + 1]
        ref = brute_force_block(w.q[s:e], w.k[s:e], w.v[s:e], w.scale)
        np.testing.assert_allclose(out[s:e], ref, rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------
# decode semantics, split combine, pool contents
# ----------------------------------------------------------------------------

def test_decode_step_equals_last_row_of_prefill_over_extended_sequence():
    w = wl.tiny(seed=12).materialise()
    cu = np.concatenate([[0], np.cumsum(w.block_lens)])
    st = oa.DecodeState(w.k, w.v, cu, w.decode_steps)
    for t in range(3):
        st.append(w.k_dec[t], w.v_dec[t])
        got = st.decode(w.q_dec[t], w.scale)
        for b in range(w.num_blocks):
            s, e = cu[b], cu[b + 1]
            qx = np.concatenate([w.q[s:e], w.q_dec[: t + 1, b]])
            kx = np.concatenate([w.k[s:e], w.k_dec[: t + 1, b]])
            vx = np.concatenate([w.v[s:e], w.v_dec[: t + 1, b]])
            ref = brute_force_block(qx, kx, vx, w.scale)[-1]
            np.testing.assert_allclose(got[b], ref, rtol=1e-11, atol=1e-13)


def test_split_combine_equals_unsplit():
    rng = np.random.default_rng(13)
    n, d = 300, 16
    q = rand_bits(rng, (1, d))
    k = rand_bits(rng, (n, 1, d))
    v = rand_bits(rng, (n, 1, d))
    k[123, 0] = bf(oa.bf16_bits_to_f64(q)[0] * 6)      # large max in one split
    whole = oa.attend_token(q, k, v, 0.25)[0]
    qf, kf, vf = oa.bf16_bits_to_f64(q)[0], oa.bf16_bits_to_f64(k)[:, 0], oa.bf16_bits_to_f64(v)[:, 0]
    for cuts in ([0, 300], [0, 1, 300], [0, 64, 128, 192, 256, 300], [0, 100, 100, 300]):
        parts = [oa.split_partial(qf, kf[a:b], vf[a:b], 0.25) for a, b in zip(cuts[:-1], cuts[1:])]
        parts.append(oa.split_partial(qf, kf[:0], vf[:0], 0.25))      # an empty split
        merged = oa.combine_splits(*zip(*parts))
        np.testing.assert_allclose(merged, whole, rtol=1e-12, atol=1e-14)


def test_expected_pool_places_tokens_by_slot():
    w = wl.custom([5, 3], 2, 2, 4, steps=2, seed=14).materialise()
    plan = op.build_plan([5, 3], 2, 4, [7, 2, 9, 4, 1], 2, 2, 1)
    kp, vp, written = oa.expected_pool(plan["slot_mapping"], w.k, w.v, 10, 4)
    assert written.sum() == 8
    np.testing.assert_array_equal(kp[7, :, 0, :], w.k[0])     # block 0, pos 0 -> page 7 offset 0
    np.testing.assert_array_equal(kp[2, :, 0, :], w.k[4])     # block 0, pos 4 -> page 2 offset 0
    np.testing.assert_array_equal(vp[9, :, 2, :], w.v[7])     # block 1, pos 2 -> page 9 offset 2
    assert not written[4].any() and not written[1].any()


# ----------------------------------------------------------------------------
# plan oracle: the paper's partition rule and a hand-worked page table
# ----------------------------------------------------------------------------

def _read_golden(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            rows.setdefault(key, []).append([int(x) for x in vals])
    return rows


def test_partition_matches_paper_worker_counts():
    with open(os.path.join(GOLDEN, "worker_counts.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            tau, block, workers = (int(x) for x in line.split())
            lens = op.partition(tau, block)
            assert len(lens) == workers and sum(lens) == tau
    lens = op.partition(100000, 16384)        # ragged last block
    assert lens == [16384] * 6 + [100000 - 6 * 16384]


def test_plan_matches_hand_worked_fixture():
    g = {k: v[0] for k, v in _read_golden("plan_small.txt").items()}
    plan = op.build_plan([5, 3], 2, 4, [7, 2, 9, 4, 1], 2, 2, 1)
    for key in ("cu_seqlens", "page_indptr", "page_indices", "slot_mapping", "split_indptr"):
        assert plan[key] == g[key], key
    assert sum(plan["prefill_items"], []) == g["prefill_items"]
    assert sum(plan["decode_items"], []) == g["decode_items"]
    assert plan["seq_lens"] == [0, 0]


def test_plan_invariants_on_ragged_lengths():
    w = wl.ragged(seed=21, num_blocks=9, lo=10, hi=700, steps=33)
    rng = np.random.default_rng(0)
    free = rng.permutation(w.num_pages).tolist()
    P, C, M = 16, 4, 128
    plan = op.build_plan(w.block_lens.tolist(), 33, P, free, 8, M, C)
    # pages are taken in order from the free list, each used once
    assert plan["page_indices"] == free[: plan["page_indptr"][-1]]
    assert len(set(plan["slot_mapping"])) == w.total_tokens
    # slot_of agrees with slot_mapping and stays inside the block's pages
    tok = 0
    for b, L in enumerate(w.block_lens):
        pages = set(plan["page_indices"][plan["page_indptr"][b]:plan["page_indptr"][b + 1]])
        assert len(pages) == -(-(int(L) + 33) // P)
        for p in range(int(L)):
            s = plan["slot_mapping"][tok]
            assert s == op.slot_of(plan, P, b, p) and s // P in pages
            tok += 1
    # every (block, tile) exactly once, costs non-increasing
    items = [tuple(x) for x in plan["prefill_items"]]
    want = {(b, t) for b, L in enumerate(w.block_lens) for t in range(-(-int(L) // M))}
    assert set(items) == want and len(items) == len(want)
    costs = [min((t + 1) * M, int(w.block_lens[b])) for b, t in items]
    assert costs == sorted(costs, reverse=True)
    # decode splits tile each block's pages exactly once per kv head
    seen = {}
    for b, g, s in plan["decode_items"]:
        seen.setdefault((b, g), []).append(s)
    for b in range(w.num_blocks):
        n_pages = plan["page_indptr"][b + 1] - plan["page_indptr"][b]
        for g in range(8):
            assert sorted(seen[(b, g)]) == list(range(-(-n_pages // C)))
        assert plan["split_indptr"][b + 1] - plan["split_indptr"][b] == -(-n_pages // C)


def test_plan_rejects_bad_input():
    with pytest.raises(ValueError):
        op.build_plan([4, 0], 1, 16, list(range(10)), 1, 128, 4)
    with pytest.raises(MemoryError):
        op.build_plan([40, 40], 8, 16, list(range(5)), 1, 128, 4)
