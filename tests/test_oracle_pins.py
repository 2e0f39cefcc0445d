"""Pins for the CPU fp64 oracle: everything here checks oracle/s2a_oracle.c against
something other than itself (the paper's printed example, an independent
transcription of Algorithm 1 with autograd, brute-force loops, closed forms,
finite differences, dependency structure).  No GPU, no CUDA library.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import algorithm1_torch as alg1
from oracle import s2a_oracle as orc
from paper_2309_12307_b200.inputs import make_inputs, make_inputs_f64

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- P1
def _read_ranges(path):
    """golden file lines: <name> <head-half> <first..last> [<first..last> ...] (1-based, inclusive)"""
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, half, *ranges = line.split()
            toks = []
            for r in ranges:
                a, b = r.split("..")
                toks.extend(range(int(a), int(b) + 1))
            out[name] = (half, toks)
    return out


def test_group_membership_matches_papers_worked_example():
    """Section 3.2: N=8192, G=2048.  Pattern 1: first group = tokens 1..2048.  Pattern 2: first
    group = 1025..3072, and the first and last 1024 tokens share a group (1-based)."""
    N, G, H = 8192, 2048, 32
    gold = _read_ranges(os.path.join(GOLDEN, "group_membership_sec3_2.txt"))
    for name, (half, toks_1based) in gold.items():
        h = 0 if half == "pattern1" else H - 1
        want = sorted(t - 1 for t in toks_1based)
        # the last member of a group (in rolled order) attends the whole group: |A| = G
        full = [orc.attended(N, H, G, h, t) for t in want if len(orc.attended(N, H, G, h, t)) == G]
        assert len(full) == 1, name
        assert sorted(full[0]) == want, name
        # and every member's attended set lies inside the group
        for t in want[:: max(1, len(want) // 64)]:
            assert set(orc.attended(N, H, G, h, t)) <= set(want)


def test_wrapped_group_order_is_tail_then_head():
    """Roll by -G/2 puts original token G/2 at rolled position 0, so the wrapped last group is
    [N-G/2, N) followed by [0, G/2): a front token attends every tail token plus its own prefix."""
    N, G, H = 32, 8, 4
    assert orc.attended(N, H, G, 3, 0) == [28, 29, 30, 31, 0]
    assert orc.attended(N, H, G, 3, 3) == [28, 29, 30, 31, 0, 1, 2, 3]
    assert orc.attended(N, H, G, 3, 4) == [4]
    assert orc.attended(N, H, G, 3, 28) == [28]
    assert orc.attended(N, H, G, 0, 28) == [24, 25, 26, 27, 28]
    assert orc.attended(N, H, G, 1, 7) == list(range(8))


# --------------------------------------------------------------------------- P2
SHAPES_P2 = [
    # B, N, G, H, Hkv, d
    (1, 16, 8, 2, 2, 4),
    (2, 16, 8, 4, 4, 3),
    (2, 32, 8, 4, 2, 5),
    (1, 24, 12, 8, 2, 4),
    (1, 64, 16, 4, 1, 8),
    (1, 16, 16, 2, 2, 4),  # one group: the shifted heads wrap the whole sequence
]


@pytest.mark.parametrize("B,N,G,H,Hkv,d", SHAPES_P2)
def test_index_form_equals_algorithm1_transcription(B, N, G, H, Hkv, d):
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=3)
    o_ref, lse_ref = alg1.s2_attn(q, k, v, G)
    dq_ref, dk_ref, dv_ref = alg1.s2_attn_grads(q, k, v, dO, G)
    o, lse = orc.fwd(q, k, v, G)
    dq, dk, dv = orc.bwd(q, k, v, dO, G)
    np.testing.assert_allclose(o, o_ref.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dq, dq_ref.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(dk, dk_ref.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(dv, dv_ref.numpy(), rtol=0, atol=1e-11)


def test_row_lists_equal_full_run():
    B, N, G, H, Hkv, d = 2, 32, 8, 4, 2, 5
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=5)
    o, lse = orc.fwd(q, k, v, G)
    dq, dk, dv = orc.bwd(q, k, v, dO, G)
    q_rows = [(b, h, t) for b in range(B) for h in range(H) for t in (0, 3, 4, 17, 31)]
    kv_rows = [(b, hk, t) for b in range(B) for hk in range(Hkv) for t in (0, 5, 12, 28, 31)]
    o_s, lse_s = orc.fwd(q, k, v, G, rows=q_rows)
    dq_s, dk_s, dv_s = orc.bwd(q, k, v, dO, G, q_rows=q_rows, kv_rows=kv_rows)
    for i, (b, h, t) in enumerate(q_rows):
        np.testing.assert_array_equal(o_s[i], o[b, t, h])
        assert lse_s[i] == lse[b, h, t]
        np.testing.assert_array_equal(dq_s[i], dq[b, t, h])
    for i, (b, hk, t) in enumerate(kv_rows):
        np.testing.assert_array_equal(dk_s[i], dk[b, t, hk])
        np.testing.assert_array_equal(dv_s[i], dv[b, t, hk])


def test_bf16_inputs_are_widened_exactly():
    B, N, G, H, Hkv, d = 1, 32, 16, 4, 2, 8
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=0)
    o_b, lse_b = orc.fwd(q, k, v, G)
    o_d, lse_d = orc.fwd(q.double(), k.double(), v.double(), G)
    np.testing.assert_array_equal(o_b, o_d)
    np.testing.assert_array_equal(lse_b, lse_d)
    g_b = orc.bwd(q, k, v, dO, G)
    g_d = orc.bwd(q.double(), k.double(), v.double(), dO.double(), G)
    for a, b in zip(g_b, g_d):
        np.testing.assert_array_equal(a, b)


# --------------------------------------------------------------------------- P3
def _full_causal_attention(q, k, v, scale):
    """Textbook causal attention on [n, d] matrices (one head), library routines only."""
    n = q.shape[0]
    s = (q @ k.T) * scale
    s = s.masked_fill(torch.ones(n, n, dtype=torch.bool).triu(1), float("-inf"))
    return torch.softmax(s, dim=-1) @ v, torch.logsumexp(s, dim=-1)


def test_single_group_no_shift_is_full_causal_attention():
    """G = N and no shifted head: the operator is ordinary causal attention (what the fine-tuned
    model uses at inference)."""
    B, N, H, Hkv, d = 1, 48, 4, 4, 8
    q, k, v, _ = make_inputs_f64(B, N, H, Hkv, d, seed=1)
    o, lse = orc.fwd(q, k, v, G=N, n_unshifted=H, shift=0)
    for h in range(H):
        o_ref, lse_ref = _full_causal_attention(q[0, :, h], k[0, :, h], v[0, :, h], 1 / math.sqrt(d))
        np.testing.assert_allclose(o[0, :, h], o_ref.numpy(), atol=1e-12)
        np.testing.assert_allclose(lse[0, h], lse_ref.numpy(), atol=1e-12)


def test_sdpa_third_opinion_on_unshifted_heads():
    """Unshifted heads equal causal attention applied to each slice [gG, (g+1)G) separately
    (checked against the library's scaled_dot_product_attention in fp64)."""
    B, N, G, H, Hkv, d = 2, 64, 16, 4, 4, 8
    q, k, v, _ = make_inputs_f64(B, N, H, Hkv, d, seed=2)
    o, _ = orc.fwd(q, k, v, G)
    for b, h, g in itertools.product(range(B), range(H // 2), range(N // G)):
        sl = slice(g * G, (g + 1) * G)
        ref = torch.nn.functional.scaled_dot_product_attention(
            q[b, sl, h][None, None], k[b, sl, h][None, None], v[b, sl, h][None, None], is_causal=True)[0, 0]
        np.testing.assert_allclose(o[b, sl, h], ref.numpy(), atol=1e-12)


def test_shifted_heads_equal_causal_attention_on_rolled_slices():
    """Shifted heads: causal attention over original tokens [gG+G/2, (g+1)G+G/2) mod N, in that order."""
    B, N, G, H, Hkv, d = 1, 64, 16, 4, 4, 8
    q, k, v, _ = make_inputs_f64(B, N, H, Hkv, d, seed=4)
    o, lse = orc.fwd(q, k, v, G)
    for h, g in itertools.product(range(H // 2, H), range(N // G)):
        idx = torch.tensor([(g * G + G // 2 + x) % N for x in range(G)])
        o_ref, lse_ref = _full_causal_attention(q[0, idx, h], k[0, idx, h], v[0, idx, h], 1 / math.sqrt(d))
        np.testing.assert_allclose(o[0, idx.numpy(), h], o_ref.numpy(), atol=1e-12)
        np.testing.assert_allclose(lse[0, h, idx.numpy()], lse_ref.numpy(), atol=1e-12)


# --------------------------------------------------------------------------- P4
def _brute_force(q, k, v, dO, G, scale):
    """Explicit Python loops written from the paper's prose: build the rolled sequence of every
    head, cut it in groups, let each member look at the members before it."""
    B, N, H, d = q.shape
    Hkv = k.shape[2]
    rep = H // Hkv
    o = np.zeros((B, N, H, d))
    dq = np.zeros((B, N, H, d))
    dk = np.zeros((B, N, Hkv, d))
    dv = np.zeros((B, N, Hkv, d))
    for b in range(B):
        for h in range(H):
            hk = h // rep
            order = list(range(N))
            if h >= H // 2:  # tokens rolled by -G/2: position p now holds token p + G/2
                order = order[G // 2:] + order[: G // 2]
            for g0 in range(0, N, G):
                members = order[g0: g0 + G]
                for x, t in enumerate(members):
                    keys = members[: x + 1]
                    z = [scale * sum(q[b, t, h, c] * k[b, u, hk, c] for c in range(d)) for u in keys]
                    zsum = sum(math.exp(zz) for zz in z)
                    p = [math.exp(zz) / zsum for zz in z]
                    for c in range(d):
                        o[b, t, h, c] = sum(pi * v[b, u, hk, c] for pi, u in zip(p, keys))
                    Dt = sum(dO[b, t, h, c] * o[b, t, h, c] for c in range(d))
                    for pi, u in zip(p, keys):
                        dp = sum(dO[b, t, h, c] * v[b, u, hk, c] for c in range(d))
                        ds = pi * (dp - Dt)
                        for c in range(d):
                            dv[b, u, hk, c] += pi * dO[b, t, h, c]
                            dq[b, t, h, c] += scale * ds * k[b, u, hk, c]
                            dk[b, u, hk, c] += scale * ds * q[b, t, h, c]
    return o, dq, dk, dv


@pytest.mark.parametrize("B,N,G,H,Hkv,d", [(1, 16, 8, 4, 4, 3), (2, 24, 6, 4, 2, 2), (1, 32, 8, 2, 1, 4)])
def test_brute_force_loops(B, N, G, H, Hkv, d):
    q, k, v, dO = (x.numpy() for x in make_inputs_f64(B, N, H, Hkv, d, seed=7))
    scale = 1 / math.sqrt(d)
    o_ref, dq_ref, dk_ref, dv_ref = _brute_force(q, k, v, dO, G, scale)
    o, _ = orc.fwd(q, k, v, G)
    dq, dk, dv = orc.bwd(q, k, v, dO, G)
    np.testing.assert_allclose(o, o_ref, atol=1e-12)
    np.testing.assert_allclose(dq, dq_ref, atol=1e-12)
    np.testing.assert_allclose(dk, dk_ref, atol=1e-12)
    np.testing.assert_allclose(dv, dv_ref, atol=1e-12)


# --------------------------------------------------------------------------- P5
def test_closed_forms():
    B, N, G, H, Hkv, d = 1, 64, 16, 4, 2, 8
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=11)
    scale = 1 / math.sqrt(d)
    o, lse = orc.fwd(q, k, v, G)
    rep = H // Hkv
    # the first member of every group attends only itself
    for h in range(H):
        s = 0 if h < H // 2 else G // 2
        for g in range(N // G):
            t = (g * G + s) % N
            np.testing.assert_allclose(o[0, t, h], v[0, t, h // rep].numpy(), atol=1e-13)
            assert abs(lse[0, h, t] - scale * float(q[0, t, h] @ k[0, t, h // rep])) < 1e-12
    # q = 0: uniform weights -> mean of the attended values, lse = ln |A|
    o0, lse0 = orc.fwd(torch.zeros_like(q), k, v, G)
    for h, t in [(0, 0), (0, 15), (1, 37), (2, 0), (3, 5), (2, 8), (3, 63), (2, 40)]:
        A = orc.attended(N, H, G, h, t)
        np.testing.assert_allclose(o0[0, t, h], v[0, A, h // rep].mean(0).numpy(), atol=1e-13)
        assert abs(lse0[0, h, t] - math.log(len(A))) < 1e-13
    # shifted head, token 0: mean over the last G/2 tokens and token 0; lse = ln(G/2 + 1)
    A0 = list(range(N - G // 2, N)) + [0]
    np.testing.assert_allclose(o0[0, 0, H - 1], v[0, A0, Hkv - 1].mean(0).numpy(), atol=1e-13)
    assert abs(lse0[0, H - 1, 0] - math.log(G // 2 + 1)) < 1e-13
    # identical value rows -> output equals that row
    c = torch.linspace(-1, 1, d, dtype=torch.float64)
    oc, _ = orc.fwd(q, k, c.expand_as(v).contiguous(), G)
    np.testing.assert_allclose(oc, np.broadcast_to(c.numpy(), oc.shape), atol=1e-13)


def test_gradient_identities():
    """Sum_t' P = 1 gives sum_t' dV[t'] = sum_{h,t} dO[t,h]; sum_t' dS = 0 gives sum_t' dK[t'] = 0
    when all q rows are equal; dQ.q summed equals dK.k summed (both are sum dS*z)."""
    B, N, G, H, Hkv, d = 2, 32, 8, 4, 2, 4
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=13)
    dq, dk, dv = orc.bwd(q, k, v, dO, G)
    rep = H // Hkv
    for b, hk in itertools.product(range(B), range(Hkv)):
        want = dO[b, :, hk * rep:(hk + 1) * rep].sum(dim=(0, 1)).numpy()
        np.testing.assert_allclose(dv[b, :, hk].sum(0), want, atol=1e-12)
        lhs = (dq[b, :, hk * rep:(hk + 1) * rep] * q[b, :, hk * rep:(hk + 1) * rep].numpy()).sum()
        rhs = (dk[b, :, hk] * k[b, :, hk].numpy()).sum()
        assert abs(lhs - rhs) < 1e-11
    q_same = q[:, :1].expand_as(q).contiguous()
    _, dk2, _ = orc.bwd(q_same, k, v, dO, G)
    # with identical q rows inside one head, sum over keys of dK = scale * q * sum dS = 0 per head;
    # with one query head per KV head the sum over t' of dK vanishes
    q1, k1, v1, dO1 = make_inputs_f64(1, 32, 2, 2, 4, seed=14)
    q1 = q1[:, :1].expand_as(q1).contiguous()
    _, dk1, _ = orc.bwd(q1, k1, v1, dO1, 8)
    np.testing.assert_allclose(dk1.sum(1), 0, atol=1e-12)


# --------------------------------------------------------------------------- P6
@pytest.mark.parametrize("Hkv", [4, 2])
def test_finite_differences(Hkv):
    B, N, G, H, d = 1, 16, 8, 4, 4
    q, k, v, dO = (x.numpy() for x in make_inputs_f64(B, N, H, Hkv, d, seed=17))
    dq, dk, dv = orc.bwd(q, k, v, dO, G)

    def loss(q_, k_, v_):
        o, _ = orc.fwd(q_, k_, v_, G)
        return float((o * dO).sum())

    eps = 1e-5
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = x[idx]
            x[idx] = old + eps
            lp = loss(q, k, v)
            x[idx] = old - eps
            lm = loss(q, k, v)
            x[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        rel = np.linalg.norm(num - grad) / np.linalg.norm(grad)
        assert rel < 1e-7, (name, rel)


# --------------------------------------------------------------------------- P7
def test_dependency_structure_and_leak_is_kept():
    """Perturbing token u changes o[t,h] iff u is in A(t,h).  Unshifted heads never see across
    group boundaries, shifted heads do, and in shifted heads the first G/2 tokens depend on the
    last G/2 tokens (the wrapped group; the default method keeps this, Fig. 3 caption / App. B)."""
    B, N, G, H, Hkv, d = 1, 32, 8, 4, 4, 4
    q, k, v, _ = make_inputs_f64(B, N, H, Hkv, d, seed=19)
    o, _ = orc.fwd(q, k, v, G)
    for u in (0, 5, 8, 12, 29, 31):
        k2, v2 = k.clone(), v.clone()
        k2[0, u] += 0.5
        v2[0, u] -= 0.25
        o2, _ = orc.fwd(q, k2, v2, G)
        changed = np.abs(o2 - o).max(axis=-1)[0] > 1e-9  # [N, H]
        for h in range(H):
            for t in range(N):
                assert changed[t, h] == (u in orc.attended(N, H, G, h, t)), (u, t, h)
    # the leak: token 2 of a shifted head depends on token N-1
    assert (N - 1) in orc.attended(N, H, G, H - 1, 2)
    # unshifted: token 8 (first of group 1) does not see token 7
    assert 7 not in orc.attended(N, H, G, 0, 8)
    # shifted: token 8 sees token 7
    assert 7 in orc.attended(N, H, G, H - 1, 8)


# --------------------------------------------------------------------------- P8
def test_gqa_equals_mha_on_repeated_kv():
    B, N, G, H, Hkv, d = 2, 32, 8, 8, 2, 4
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=23)
    rep = H // Hkv
    kr, vr = k.repeat_interleave(rep, dim=2), v.repeat_interleave(rep, dim=2)
    o_g, lse_g = orc.fwd(q, k, v, G)
    o_m, lse_m = orc.fwd(q, kr, vr, G)
    np.testing.assert_allclose(o_g, o_m, atol=1e-13)
    np.testing.assert_allclose(lse_g, lse_m, atol=1e-13)
    dq_g, dk_g, dv_g = orc.bwd(q, k, v, dO, G)
    dq_m, dk_m, dv_m = orc.bwd(q, kr, vr, dO, G)
    np.testing.assert_allclose(dq_g, dq_m, atol=1e-12)
    np.testing.assert_allclose(dk_g, dk_m.reshape(B, N, Hkv, rep, d).sum(3), atol=1e-12)
    np.testing.assert_allclose(dv_g, dv_m.reshape(B, N, Hkv, rep, d).sum(3), atol=1e-12)


def test_planted_mistakes_are_caught():
    """The pins must be able to fail: a wrong shift amount, a dropped scale or an
    unshifted second half each move the result."""
    B, N, G, H, Hkv, d = 1, 32, 8, 4, 4, 4
    q, k, v, _ = make_inputs_f64(B, N, H, Hkv, d, seed=29)
    o, _ = orc.fwd(q, k, v, G)
    # rolling by +G/2 instead of -G/2 gives the SAME partition (boundaries at G/2 + multiples of G,
    # same in-group order), so the direction cannot matter (App. B, variant 1) ...
    o_other_dir, _ = orc.fwd(q, k, v, G, shift=-(G // 2))
    np.testing.assert_array_equal(o, o_other_dir)
    # ... but a wrong amount does
    o_quarter, _ = orc.fwd(q, k, v, G, shift=G // 4)
    assert np.abs(o - o_quarter).max() > 1e-3
    o_noscale, _ = orc.fwd(q, k, v, G, scale=1.0)
    assert np.abs(o - o_noscale).max() > 1e-3
    o_noshift, _ = orc.fwd(q, k, v, G, n_unshifted=H)
    assert np.abs(o - o_noshift)[:, :, H // 2:].max() > 1e-3
    np.testing.assert_array_equal(o[:, :, : H // 2], o_noshift[:, :, : H // 2])


# --------------------------------------------------------------------------- P9
def test_flop_accounting_matches_papers_table():
    """Table 11 (FLOPs profiling): attention FLOPs of Llama2-7B (32 layers, 32 heads, d=128),
    non-causal count with 2 FLOPs per multiply-add; S2-Attn at G=N/4 costs a quarter."""
    rows = []
    with open(os.path.join(GOLDEN, "flops_table11.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                n, full, s2 = line.split()
                rows.append((int(n), float(full), float(s2)))
    assert len(rows) == 4
    L, H, d = 32, 32, 128
    for N, full_T, s2_T in rows:
        G = N // 4
        full = 4 * N * N * d * H * L / 1e12
        s2 = 4 * N * G * d * H * L / 1e12
        assert abs(full - full_T) <= 0.051, (N, full)
        assert abs(s2 - s2_T) <= 0.051, (N, s2)
    # the benchmark's metric counts only the causal in-group pairs: G(G+1)/2 per (b, h, group)
    from paper_2309_12307_b200.inputs import WORKLOADS
    w = WORKLOADS["llama2_7b_32k"]
    assert w.pairs == 4_295_491_584
    assert abs(w.flops_fwd_bwd / 1e12 - 7.698) < 1e-3
    # and the count equals the sizes of the attended sets
    N, G, H = 32, 8, 4
    assert sum(len(orc.attended(N, H, G, h, t)) for h in range(H) for t in range(N)) == H * (N // G) * G * (G + 1) // 2


# --------------------------------------------------------------------------- variant 2 (Appendix B)
@pytest.mark.parametrize("B,N,G,H,Hkv,d", [(1, 16, 8, 2, 2, 4), (2, 32, 8, 4, 2, 5), (1, 16, 16, 2, 1, 4)])
def test_leak_free_variant_equals_masked_transcription(B, N, G, H, Hkv, d):
    """Variant 2: the wrapped group of the shifted heads is cut at the wrap.  Index form against the
    Algorithm-1 transcription with the extra mask, forward and autograd backward."""
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=31)
    o_ref, lse_ref = alg1.s2_attn(q, k, v, G, leak_free=True)
    dq_ref, dk_ref, dv_ref = alg1.s2_attn_grads(q, k, v, dO, G, leak_free=True)
    o, lse = orc.fwd(q, k, v, G, leak_free=True)
    dq, dk, dv = orc.bwd(q, k, v, dO, G, leak_free=True)
    np.testing.assert_allclose(o, o_ref.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dq, dq_ref.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(dk, dk_ref.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(dv, dv_ref.numpy(), rtol=0, atol=1e-11)


def test_leak_free_variant_removes_exactly_the_leak():
    """With variant 2 the first G/2 tokens of a shifted head are plain causal attention over
    themselves, the last G/2 tokens likewise, and every other row equals the default method."""
    B, N, G, H, Hkv, d = 1, 64, 16, 4, 4, 8
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=37)
    o_def, _ = orc.fwd(q, k, v, G)
    o_v2, lse_v2 = orc.fwd(q, k, v, G, leak_free=True)
    half = G // 2
    for h in range(H // 2, H):
        for sl in (slice(0, half), slice(N - half, N)):
            o_ref, lse_ref = _full_causal_attention(q[0, sl, h], k[0, sl, h], v[0, sl, h], 1 / math.sqrt(d))
            np.testing.assert_allclose(o_v2[0, sl, h], o_ref.numpy(), atol=1e-12)
            np.testing.assert_allclose(lse_v2[0, h, sl], lse_ref.numpy(), atol=1e-12)
    # only the front tokens of the shifted heads change
    changed = np.abs(o_v2 - o_def).max(axis=-1)[0] > 1e-12     # [N, H]
    assert not changed[:, : H // 2].any()
    assert not changed[half:, H // 2:].any()
    assert changed[:half, H // 2:].all()
    # and they no longer depend on the tail tokens
    k2, v2 = k.clone(), v.clone()
    k2[0, N - 3] += 1.0
    v2[0, N - 3] -= 1.0
    o_pert, _ = orc.fwd(q, k2, v2, G, leak_free=True)
    assert np.abs(o_pert - o_v2)[0, :half].max() == 0.0
    # gradients: finite differences on one coordinate of each input
    dq, dk, dv = orc.bwd(q, k, v, dO, G, leak_free=True)
    eps = 1e-6
    for x, grad, idx in ((q, dq, (0, 2, 3, 1)), (k, dk, (0, N - 2, 3, 0)), (v, dv, (0, 1, 2, 5))):
        xp, xm = x.clone(), x.clone()
        xp[idx] += eps
        xm[idx] -= eps
        args_p = [xp if t is x else t for t in (q, k, v)]
        args_m = [xm if t is x else t for t in (q, k, v)]
        lp = (orc.fwd(*args_p, G, leak_free=True)[0] * dO.numpy()).sum()
        lm = (orc.fwd(*args_m, G, leak_free=True)[0] * dO.numpy()).sum()
        assert abs((lp - lm) / (2 * eps) - grad[idx]) < 1e-6


# --------------------------------------------------------------------------- variant 3 (Appendix B)
@pytest.mark.parametrize("B,N,G,H,Hkv,d", [(1, 16, 8, 2, 2, 4), (2, 32, 8, 4, 2, 5), (1, 16, 16, 2, 1, 4)])
def test_swapped_variant_equals_swapped_transcription(B, N, G, H, Hkv, d):
    """Variant 3: the two halves of the wrapped group of the shifted heads change places.  Index form
    against the Algorithm-1 transcription that really swaps the tokens (and swaps back), forward and
    autograd backward."""
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=41)
    o_ref, lse_ref = alg1.s2_attn(q, k, v, G, swap_wrapped=True)
    dq_ref, dk_ref, dv_ref = alg1.s2_attn_grads(q, k, v, dO, G, swap_wrapped=True)
    o, lse = orc.fwd(q, k, v, G, swap_wrapped=True)
    dq, dk, dv = orc.bwd(q, k, v, dO, G, swap_wrapped=True)
    np.testing.assert_allclose(o, o_ref.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lse_ref.numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(dq, dq_ref.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(dk, dk_ref.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(dv, dv_ref.numpy(), rtol=0, atol=1e-11)


def test_swapped_variant_is_causal_attention_in_original_token_order():
    """With variant 3 the wrapped group of a shifted head is plain causal attention over its tokens
    taken in original order: the first G/2 tokens of the sequence, then the last G/2.  So no token
    attends a later one any more, and every other row equals the default method."""
    B, N, G, H, Hkv, d = 1, 64, 16, 4, 4, 8
    q, k, v, dO = make_inputs_f64(B, N, H, Hkv, d, seed=43)
    o_def, _ = orc.fwd(q, k, v, G)
    o_v3, lse_v3 = orc.fwd(q, k, v, G, swap_wrapped=True)
    half = G // 2
    members = list(range(0, half)) + list(range(N - half, N))
    for h in range(H // 2, H):
        o_ref, lse_ref = _full_causal_attention(q[0, members, h], k[0, members, h], v[0, members, h], 1 / math.sqrt(d))
        np.testing.assert_allclose(o_v3[0, members, h], o_ref.numpy(), atol=1e-12)
        np.testing.assert_allclose(lse_v3[0, h, members], lse_ref.numpy(), atol=1e-12)
    # only the wrapped group of the shifted heads changes (token 0 attends itself alone either way? no:
    # by default it attends the tail as well, so all G tokens of the group change)
    changed = np.abs(o_v3 - o_def).max(axis=-1)[0] > 1e-12     # [N, H]
    assert not changed[:, : H // 2].any()
    assert not changed[half:N - half, H // 2:].any()
    assert changed[members][:, H // 2:].all()
    # causality in original order: perturbing token t changes no output before t (any head)
    for t_pert in (3, N - 3):
        k2, v2 = k.clone(), v.clone()
        k2[0, t_pert] += 1.0
        v2[0, t_pert] -= 1.0
        o_pert, _ = orc.fwd(q, k2, v2, G, swap_wrapped=True)
        assert np.abs(o_pert - o_v3)[0, :t_pert].max() == 0.0
    # ... which the default method violates (the leak): token 1 of a shifted head sees token N-3
    k2, v2 = k.clone(), v.clone()
    k2[0, N - 3] += 1.0
    o_pert, _ = orc.fwd(q, k2, v2, G)
    assert np.abs(o_pert - o_def)[0, 1, H // 2:].max() > 0.0
    # gradients: finite differences on one coordinate of each input
    dq, dk, dv = orc.bwd(q, k, v, dO, G, swap_wrapped=True)
    eps = 1e-6
    for x, grad, idx in ((q, dq, (0, N - 2, 3, 1)), (k, dk, (0, 2, 3, 0)), (v, dv, (0, N - 5, 2, 5))):
        xp, xm = x.clone(), x.clone()
        xp[idx] += eps
        xm[idx] -= eps
        args_p = [xp if t is x else t for t in (q, k, v)]
        args_m = [xm if t is x else t for t in (q, k, v)]
        lp = (orc.fwd(*args_p, G, swap_wrapped=True)[0] * dO.numpy()).sum()
        lm = (orc.fwd(*args_m, G, swap_wrapped=True)[0] * dO.numpy()).sum()
        assert abs((lp - lm) / (2 * eps) - grad[idx]) < 1e-6


def test_variants_2_and_3_exclude_each_other():
    q, k, v, _ = make_inputs_f64(1, 16, 2, 2, 4, seed=1)
    with pytest.raises(ValueError):
        orc.fwd(q, k, v, 8, leak_free=True, swap_wrapped=True)
