"""Parity of the CUDA path (through the C-ABI) against the CPU fp64 oracle, element by element on
small seeded inputs and on sampled rows at the benchmark's full sizes.

Tolerances (bf16 inputs, fp32 accumulation, bf16 outputs): max abs error 2e-2 on o, relative L2
error 1e-2 on dq, dk, dv; lse (fp32) within 2e-3.
"""
import math

import numpy as np
import pytest
import torch

from oracle import s2a_oracle as orc
from paper_2309_12307_b200.inputs import WORKLOADS, make_inputs, make_inputs_periodic

pytestmark = pytest.mark.gpu

O_ATOL = 2e-2
GRAD_REL_L2 = 1e-2
LSE_ATOL = 2e-3


@pytest.fixture(scope="module")
def s2a():
    from paper_2309_12307_b200 import binding

    binding.load()
    return binding


def rel_l2(got, want):
    got = np.asarray(got, dtype=np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))


def run_gpu(s2a, q, k, v, dO, G, **ex):
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    if ex:
        o, lse = s2a.s2a_fwd_ex(qd, kd, vd, G, **ex)
        dq, dk, dv = s2a.s2a_bwd_ex(qd, kd, vd, o, lse, dOd, G, **ex)
    else:
        o, lse = s2a.s2a_fwd(qd, kd, vd, G)
        dq, dk, dv = s2a.s2a_bwd(qd, kd, vd, o, lse, dOd, G)
    torch.cuda.synchronize()
    rc, where = s2a.device_status()
    assert rc == 0, f"device status {rc} at wait {where}"
    return tuple(x.float().cpu().numpy().astype(np.float64) for x in (o, lse, dq, dk, dv))


SMALL = [
    # B, N, G, H, Hkv, d      several tiles per group, wrapped groups, GQA ratios 1/2/4/8
    (1, 1024, 256, 4, 4, 64),     # the tiny benchmark configuration
    (1, 512, 256, 2, 2, 128),
    (2, 1024, 512, 4, 2, 128),
    (1, 1536, 768, 8, 2, 64),     # group = 6 tiles, not a power of two
    (1, 1024, 1024, 2, 2, 128),   # single group: the shifted head wraps the whole sequence
    (2, 512, 256, 8, 1, 128),     # one KV head shared by shifted and unshifted query heads
    (1, 2048, 1024, 16, 2, 64),   # GQA ratio 8
]


@pytest.mark.parametrize("B,N,G,H,Hkv,d", SMALL)
def test_small_shapes_match_oracle_everywhere(s2a, B, N, G, H, Hkv, d):
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=0)
    o, lse, dq, dk, dv = run_gpu(s2a, q, k, v, dO, G)
    o_ref, lse_ref = orc.fwd(q, k, v, G)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G)
    assert np.abs(o - o_ref).max() <= O_ATOL
    assert np.abs(lse - lse_ref).max() <= LSE_ATOL
    assert rel_l2(dq, dq_ref) <= GRAD_REL_L2
    assert rel_l2(dk, dk_ref) <= GRAD_REL_L2
    assert rel_l2(dv, dv_ref) <= GRAD_REL_L2
    # per-head slices too, so that one bad head cannot hide in the aggregate
    for h in range(H):
        assert rel_l2(dq[:, :, h], dq_ref[:, :, h]) <= GRAD_REL_L2, h
    for hk in range(Hkv):
        assert rel_l2(dk[:, :, hk], dk_ref[:, :, hk]) <= GRAD_REL_L2, hk
        assert rel_l2(dv[:, :, hk], dv_ref[:, :, hk]) <= GRAD_REL_L2, hk


def test_generalised_shift_and_head_split(s2a):
    """Pattern 1 only, pattern 2 only, full causal attention (G = N, nothing shifted), and a
    custom scale all match the oracle given the same parameters."""
    B, N, G, H, Hkv, d = 1, 1024, 512, 4, 2, 64
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=1)
    cases = [
        dict(n_unshifted=H, shift=0),
        dict(n_unshifted=0, shift=G // 2),
        dict(n_unshifted=1, shift=128, scale=0.2),
        dict(n_unshifted=2, shift=-(G // 2)),
        dict(leak_free=True),                               # Appendix B, variant 2
        dict(n_unshifted=1, shift=128, leak_free=True),
        dict(n_unshifted=2, shift=-(G // 2), leak_free=True),
        dict(swap_wrapped=True),                            # Appendix B, variant 3
        dict(n_unshifted=1, shift=128, swap_wrapped=True),
        dict(n_unshifted=2, shift=-(G // 2), swap_wrapped=True),
    ]
    for ex in cases:
        o, lse, dq, dk, dv = run_gpu(s2a, q, k, v, dO, G, **ex)
        o_ref, lse_ref = orc.fwd(q, k, v, G, **ex)
        dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, **ex)
        assert np.abs(o - o_ref).max() <= O_ATOL, ex
        assert np.abs(lse - lse_ref).max() <= LSE_ATOL, ex
        for got, want in ((dq, dq_ref), (dk, dk_ref), (dv, dv_ref)):
            assert rel_l2(got, want) <= GRAD_REL_L2, ex
    # full causal attention
    o, lse, dq, dk, dv = run_gpu(s2a, q, k, v, dO, N, n_unshifted=H, shift=0)
    o_ref, _ = orc.fwd(q, k, v, N, n_unshifted=H, shift=0)
    assert np.abs(o - o_ref).max() <= O_ATOL


RAGGED = [
    # B, N, G, H, Hkv, d, extra     G or G/2 not a multiple of the 128-token tile: ragged last tiles, and the
    #                               wrapped group of the shifted heads is cut into two runs of tiles
    (1, 1200, 200, 4, 4, 64, {}),       # two tiles per run (128 + 72), wrapped group 100 + 100
    (2, 2000, 1000, 4, 2, 128, {}),     # 8 tiles per group (7 x 128 + 104); wrapped group 500 + 500
    (1, 1536, 384, 4, 1, 64, dict(n_unshifted=0, shift=192)),   # MQA, every head shifted by half a tile more than one tile
    (1, 1280, 128, 2, 2, 128, {}),      # G = one tile, shift = half a tile
    (1, 640, 40, 2, 2, 64, {}),         # groups far smaller than a tile
    (1, 3000, 1000, 4, 4, 128, dict(leak_free=True)),                           # variant 2 with a ragged cut
    (1, 1200, 600, 4, 2, 64, dict(n_unshifted=2, shift=-300)),                  # other roll direction
    (1, 1200, 600, 4, 2, 64, dict(n_unshifted=2, shift=44, scale=0.3)),         # arbitrary shift (multiple of 4)
    (1, 1200, 600, 4, 2, 64, dict(n_unshifted=2, shift=44, leak_free=True)),
    (1, 904, 904, 2, 2, 64, dict(n_unshifted=2, shift=0)),                      # full causal attention, ragged length
    (1, 3000, 1000, 4, 4, 128, dict(swap_wrapped=True)),                        # variant 3 with ragged runs
    (2, 1200, 600, 4, 2, 64, dict(n_unshifted=2, shift=44, swap_wrapped=True)),
]


@pytest.mark.parametrize("B,N,G,H,Hkv,d,ex", RAGGED)
def test_ragged_group_sizes_match_oracle_everywhere(s2a, B, N, G, H, Hkv, d, ex):
    """Group sizes as the paper uses them (G = N/4 of any N, e.g. 25,000 of 100,000) need not be a
    multiple of the 128-token tile.  Outputs are pre-filled with NaN: every row must be written, by
    exactly the tile that owns it."""
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=11)
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((B, H, N), float("nan"), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.full_like(qd, float("nan")), torch.full_like(kd, float("nan")), torch.full_like(vd, float("nan"))
    if ex:
        s2a.s2a_fwd_ex(qd, kd, vd, G, o=o, lse=lse, **ex)
        s2a.s2a_bwd_ex(qd, kd, vd, o, lse, dOd, G, dq=dq, dk=dk, dv=dv, **ex)
    else:
        s2a.s2a_fwd(qd, kd, vd, G, o=o, lse=lse)
        s2a.s2a_bwd(qd, kd, vd, o, lse, dOd, G, dq=dq, dk=dk, dv=dv)
    torch.cuda.synchronize()
    assert s2a.device_status()[0] == 0
    o, lse, dq, dk, dv = (x.float().cpu().numpy().astype(np.float64) for x in (o, lse, dq, dk, dv))
    o_ref, lse_ref = orc.fwd(q, k, v, G, **ex)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, **ex)
    for x in (o, lse, dq, dk, dv):
        assert np.isfinite(x).all()
    assert np.abs(o - o_ref).max() <= O_ATOL
    assert np.abs(lse - lse_ref).max() <= LSE_ATOL
    for h in range(H):
        assert rel_l2(dq[:, :, h], dq_ref[:, :, h]) <= GRAD_REL_L2, h
    for hk in range(Hkv):
        assert rel_l2(dk[:, :, hk], dk_ref[:, :, hk]) <= GRAD_REL_L2, hk
        assert rel_l2(dv[:, :, hk], dv_ref[:, :, hk]) <= GRAD_REL_L2, hk


def test_many_small_units_sampled_rows(s2a):
    """Batch 4 x 32 heads x 4 groups of a short sequence: 512 (batch, head, group) units, i.e. many more
    units than SMs and several chunks of the block order; sampled rows against the oracle."""
    B, N, G, H, Hkv, d = 4, 4096, 1024, 32, 8, 128
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=21)
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    o, lse = s2a.s2a_fwd(qd, kd, vd, G)
    dq, dk, dv = s2a.s2a_bwd(qd, kd, vd, o, lse, dOd, G)
    torch.cuda.synchronize()
    assert s2a.device_status()[0] == 0
    rng = np.random.default_rng(3)
    q_rows = [(int(b), int(h), int(t)) for b, h, t in zip(rng.integers(0, B, 40), rng.integers(0, H, 40), rng.integers(0, N, 40))]
    q_rows += [(B - 1, H - 1, 0), (B - 1, H - 1, N - 1), (0, H // 2, G // 2), (B - 1, 0, N - 1)]
    kv_rows = [(int(b), int(h), int(t)) for b, h, t in zip(rng.integers(0, B, 24), rng.integers(0, Hkv, 24), rng.integers(0, N, 24))]
    o_ref, lse_ref = orc.fwd(q, k, v, G, rows=q_rows)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, q_rows=q_rows, kv_rows=kv_rows)
    qi = torch.tensor(q_rows, device=dev)
    ki = torch.tensor(kv_rows, device=dev)
    assert np.abs(o[qi[:, 0], qi[:, 2], qi[:, 1]].double().cpu().numpy() - o_ref).max() <= O_ATOL
    assert np.abs(lse[qi[:, 0], qi[:, 1], qi[:, 2]].double().cpu().numpy() - lse_ref).max() <= LSE_ATOL
    assert rel_l2(dq[qi[:, 0], qi[:, 2], qi[:, 1]].double().cpu().numpy(), dq_ref) <= GRAD_REL_L2
    assert rel_l2(dk[ki[:, 0], ki[:, 2], ki[:, 1]].double().cpu().numpy(), dk_ref) <= GRAD_REL_L2
    assert rel_l2(dv[ki[:, 0], ki[:, 2], ki[:, 1]].double().cpu().numpy(), dv_ref) <= GRAD_REL_L2
    assert torch.isfinite(dq.float()).all() and torch.isfinite(dk.float()).all() and torch.isfinite(dv.float()).all()


def test_tensors_of_more_than_2_31_elements(s2a):
    """B * N * H * d = 2.18e9 elements per query-side tensor (4.4 GB): every offset into q, o, dO, dq is
    computed in 64 bits or wrong.  Rows of the last batch entry, last group (the highest addresses), and of
    the first, against the oracle."""
    B, N, G, H, Hkv, d = 2, 266240, 66560, 32, 8, 128
    assert B * N * H * d > 2 ** 31
    q, k, v, dO = make_inputs_periodic(B, N, H, Hkv, d, period=4096, seed=17)
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    o, lse = s2a.s2a_fwd(qd, kd, vd, G)
    dq, dk, dv = s2a.s2a_bwd(qd, kd, vd, o, lse, dOd, G)
    torch.cuda.synchronize()
    assert s2a.device_status()[0] == 0
    q_rows = [(1, H - 1, N - 1), (1, H - 1, G // 2 - 1), (1, H // 2 - 1, N - 1), (1, 0, N - G + 5), (1, H - 1, N - G // 2 - 1),
              (0, 0, 0), (0, H - 1, G // 2), (0, 3, 70000), (1, 17, 200001)]
    # key rows near the end of their group in their head's partition (few queries attend them, so the
    # oracle stays fast): KV head 0 is unshifted, KV head Hkv-1 serves shifted query heads only
    kv_rows = [(1, 0, N - 2), (1, 0, N - 130), (0, 0, G - 1), (1, Hkv - 1, G // 2 - 3), (1, Hkv - 1, G + G // 2 - 70),
               (1, Hkv - 1, N - G // 2 - 2)]
    o_ref, lse_ref = orc.fwd(q, k, v, G, rows=q_rows)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, q_rows=q_rows, kv_rows=kv_rows)
    qi = torch.tensor(q_rows, device=dev)
    ki = torch.tensor(kv_rows, device=dev)
    assert np.abs(o[qi[:, 0], qi[:, 2], qi[:, 1]].double().cpu().numpy() - o_ref).max() <= O_ATOL
    assert np.abs(lse[qi[:, 0], qi[:, 1], qi[:, 2]].double().cpu().numpy() - lse_ref).max() <= LSE_ATOL
    assert rel_l2(dq[qi[:, 0], qi[:, 2], qi[:, 1]].double().cpu().numpy(), dq_ref) <= GRAD_REL_L2
    assert rel_l2(dk[ki[:, 0], ki[:, 2], ki[:, 1]].double().cpu().numpy(), dk_ref) <= GRAD_REL_L2
    assert rel_l2(dv[ki[:, 0], ki[:, 2], ki[:, 1]].double().cpu().numpy(), dv_ref) <= GRAD_REL_L2
    # the first member of every group attends only itself: o = v there, in the last batch entry too
    t_first = torch.tensor([(g * G + G // 2) % N for g in range(N // G)], device=dev)
    assert torch.equal(o[1, t_first, H - 1], vd[1, t_first, Hkv - 1])
    del qd, kd, vd, dOd, o, lse, dq, dk, dv
    torch.cuda.empty_cache()


def test_leak_free_variant_matches_oracle(s2a):
    """Appendix B, variant 2 on a head-dim-128 GQA shape with eight tiles per group: the wrapped group
    of the shifted heads is cut at the wrap (tile 4 of 8)."""
    B, N, G, H, Hkv, d = 2, 2048, 1024, 4, 2, 128
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=5)
    o, lse, dq, dk, dv = run_gpu(s2a, q, k, v, dO, G, leak_free=True)
    o_ref, lse_ref = orc.fwd(q, k, v, G, leak_free=True)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, leak_free=True)
    assert np.abs(o - o_ref).max() <= O_ATOL
    assert np.abs(lse - lse_ref).max() <= LSE_ATOL
    for got, want in ((dq, dq_ref), (dk, dk_ref), (dv, dv_ref)):
        assert rel_l2(got, want) <= GRAD_REL_L2
    # the variant changes only the first G/2 tokens of the shifted heads
    o_def, _, _, _, _ = run_gpu(s2a, q, k, v, dO, G)
    assert np.array_equal(o[:, G // 2:], o_def[:, G // 2:])
    assert np.array_equal(o[:, :, : H // 2], o_def[:, :, : H // 2])
    assert np.abs(o[:, : G // 2, H // 2:] - o_def[:, : G // 2, H // 2:]).max() > 1e-3


@pytest.mark.parametrize("B,N,G,H,d", [(2, 1024, 512, 4, 128), (1, 1200, 200, 4, 64)])
def test_packed_qkv_equals_separate_tensors(s2a, B, N, G, H, d):
    """Algorithm 1 takes qkv packed as [B, N, 3, H, d]; the packed entry points must give exactly
    what the separate-tensor entry points give on the same values (only strides differ).  The
    second shape has ragged tiles (G = 200)."""
    q, k, v, dO = (x.cuda() for x in make_inputs(B, N, H, H, d, seed=7))
    qkv = torch.stack([q, k, v], dim=2).contiguous()          # [B, N, 3, H, d]
    o, lse = s2a.s2a_fwd(q, k, v, G)
    dq, dk, dv = s2a.s2a_bwd(q, k, v, o, lse, dO, G)
    o_p, lse_p = s2a.s2a_fwd_packed(qkv, G)
    dqkv = torch.full_like(qkv, float("nan"))
    s2a.s2a_bwd_packed(qkv, o_p, lse_p, dO, G, dqkv=dqkv)
    torch.cuda.synchronize()
    assert torch.equal(o, o_p) and torch.equal(lse, lse_p)
    assert torch.equal(dqkv[:, :, 0], dq) and torch.equal(dqkv[:, :, 1], dk) and torch.equal(dqkv[:, :, 2], dv)


@pytest.mark.parametrize("B,N,G,H,Hkv,d", [(1, 1024, 256, 4, 4, 64), (2, 1024, 512, 8, 2, 128), (1, 1200, 200, 4, 4, 64),
                                           (1, 512, 256, 6, 3, 64)])
def test_host_buffer_entry_point_equals_device_path(s2a, B, N, G, H, Hkv, d):
    """s2a_fwd_bwd_host stages the heads through the device in chunks with its own copy streams; what
    lands in the host outputs must be exactly what s2a_fwd + s2a_bwd give on device tensors, on
    two calls in a row (the copy streams and events are reused)."""
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=13)
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    o, lse = s2a.s2a_fwd(qd, kd, vd, G)
    dq, dk, dv = s2a.s2a_bwd(qd, kd, vd, o, lse, dOd, G, fast=False)   # the host path below gets a minimum workspace too
    want = [x.cpu() for x in (o, lse, dq, dk, dv)]
    pin = [x.pin_memory() for x in (q, k, v, dO)]
    ws = torch.empty(max(s2a.bwd_workspace_bytes(B, N, H, Hkv, d, G), 256), dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream()
    for _ in range(2):
        host_out = [torch.full_like(x, float("nan")).pin_memory() for x in want]
        dev_bufs = [torch.empty_like(x) for x in (qd, kd, vd, dOd, o, lse, dq, dk, dv)]
        s2a.s2a_fwd_bwd_host(pin, host_out, dev_bufs, G, ws, stream=stream)
        stream.synchronize()
        assert s2a.device_status()[0] == 0
        for got, ref in zip(host_out, want):
            assert torch.equal(got, ref)


def test_swapped_variant_matches_oracle(s2a):
    """Appendix B, variant 3 on a head-dim-128 GQA shape with eight tiles per group: in the wrapped group
    of the shifted heads the four tiles of the sequence's front come before the four of its tail; and the
    two variant flags exclude each other."""
    B, N, G, H, Hkv, d = 2, 2048, 1024, 4, 2, 128
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=6)
    o, lse, dq, dk, dv = run_gpu(s2a, q, k, v, dO, G, swap_wrapped=True)
    o_ref, lse_ref = orc.fwd(q, k, v, G, swap_wrapped=True)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, swap_wrapped=True)
    assert np.abs(o - o_ref).max() <= O_ATOL
    assert np.abs(lse - lse_ref).max() <= LSE_ATOL
    for got, want in ((dq, dq_ref), (dk, dk_ref), (dv, dv_ref)):
        assert rel_l2(got, want) <= GRAD_REL_L2
    # it differs from the default method exactly in the wrapped group of the shifted heads
    o_def, _ = orc.fwd(q, k, v, G)
    assert np.abs(o_ref - o_def)[:, G // 2:N - G // 2].max() == 0.0
    assert np.abs(o - o_def)[:, :G // 2, H // 2:].max() > 0.1
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_fwd_ex(q.cuda(), k.cuda(), v.cuda(), G, leak_free=True, swap_wrapped=True)
    assert e.value.status == s2a.S2A_ERR_INVALID_ARG


def test_autograd_wrapper_matches_oracle(s2a):
    from paper_2309_12307_b200.autograd import s2_attn

    B, N, G, H, Hkv, d = 1, 1024, 512, 4, 2, 128
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=6)
    qd, kd, vd = (x.cuda().requires_grad_(True) for x in (q, k, v))
    o = s2_attn(qd, kd, vd, G)
    (o.float() * dO.cuda().float()).sum().backward()
    torch.cuda.synchronize()
    o_ref, _ = orc.fwd(q, k, v, G)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G)
    assert np.abs(o.detach().double().cpu().numpy() - o_ref).max() <= O_ATOL
    for got, want in ((qd.grad, dq_ref), (kd.grad, dk_ref), (vd.grad, dv_ref)):
        assert rel_l2(got.double().cpu().numpy(), want) <= GRAD_REL_L2
    # with options: variant 3 and a custom scale
    ex = dict(swap_wrapped=True, scale=0.11)
    qd, kd, vd = (x.cuda().requires_grad_(True) for x in (q, k, v))
    o = s2_attn(qd, kd, vd, G, **ex)
    (o.float() * dO.cuda().float()).sum().backward()
    torch.cuda.synchronize()
    o_ref, _ = orc.fwd(q, k, v, G, **ex)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, G, **ex)
    assert np.abs(o.detach().double().cpu().numpy() - o_ref).max() <= O_ATOL
    for got, want in ((qd.grad, dq_ref), (kd.grad, dk_ref), (vd.grad, dv_ref)):
        assert rel_l2(got.double().cpu().numpy(), want) <= GRAD_REL_L2


def test_outputs_are_deterministic_and_fully_written(s2a):
    B, N, G, H, Hkv, d = 1, 1024, 256, 4, 2, 128
    q, k, v, dO = (x.cuda() for x in make_inputs(B, N, H, Hkv, d, seed=2))
    outs = []
    for _ in range(2):
        o = torch.full_like(q, float("nan"))
        lse = torch.full((B, H, N), float("nan"), device="cuda")
        s2a.s2a_fwd(q, k, v, G, o=o, lse=lse)
        dq, dk, dv = (torch.full_like(x, float("nan")) for x in (q, k, v))
        s2a.s2a_bwd(q, k, v, o, lse, dO, G, dq=dq, dk=dk, dv=dv)
        torch.cuda.synchronize()
        outs.append((o, lse, dq, dk, dv))
    for a, b in zip(*outs):
        assert not torch.isnan(a).any()
        assert torch.equal(a, b)


def test_guard_bands_stay_intact(s2a):
    """Outputs sit inside larger buffers filled with a sentinel; nothing outside them may change."""
    B, N, G, H, Hkv, d = 1, 512, 256, 2, 2, 64
    q, k, v, dO = (x.cuda() for x in make_inputs(B, N, H, Hkv, d, seed=3))
    pad = 1024  # elements, keeps 16-byte alignment

    def guarded(shape, dtype):
        n = int(np.prod(shape))
        buf = torch.full((n + 2 * pad,), 7.0, dtype=dtype, device="cuda")
        return buf, buf[pad:pad + n].view(shape)

    bo, o = guarded(q.shape, torch.bfloat16)
    bl, lse = guarded((B, H, N), torch.float32)
    bq, dq = guarded(q.shape, torch.bfloat16)
    bk, dk = guarded(k.shape, torch.bfloat16)
    bv, dv = guarded(v.shape, torch.bfloat16)
    s2a.s2a_fwd(q, k, v, G, o=o, lse=lse)
    s2a.s2a_bwd(q, k, v, o, lse, dO, G, dq=dq, dk=dk, dv=dv)
    torch.cuda.synchronize()
    for buf in (bo, bl, bq, bk, bv):
        assert (buf[:pad] == 7.0).all() and (buf[-pad:] == 7.0).all()


def test_runtime_rejections_on_device(s2a):
    q, k, v, dO = (x.cuda() for x in make_inputs(1, 512, 2, 2, 64, seed=4))
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_fwd(*(x[:, :504].contiguous() for x in (q, k, v)), 252)   # G/2 is not a multiple of 4 tokens
    assert e.value.status == s2a.S2A_ERR_UNSUPPORTED
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_fwd_ex(q, k[:, :, :1].contiguous(), v[:, :, :1].contiguous(), 128, n_unshifted=1, shift=64)   # ragged tiles, mixed shifts on one KV head
    assert e.value.status == s2a.S2A_ERR_UNSUPPORTED
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_fwd(q, k, v, 384)          # N % G
    assert e.value.status == s2a.S2A_ERR_INVALID_ARG
    o, lse = s2a.s2a_fwd(q, k, v, 256)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_bwd(q, k, v, o, lse, dO, 256, workspace=small)
    assert e.value.status == s2a.S2A_ERR_INVALID_ARG


# ------------------------------------------------------------------------------------------------
# full benchmark sizes: sampled rows against the oracle + properties that hold at any size
# ------------------------------------------------------------------------------------------------
def _sample_rows(w, kv_tail):
    N, G, H, Hkv = w.N, w.G, w.H, w.Hkv
    rep = H // Hkv
    rng = np.random.default_rng(0)
    toks = {0, 1, 127, 128, G // 2 - 1, G // 2, G - 1, G, N - G // 2 - 1, N - G // 2, N - 1}
    toks |= set(int(t) for t in rng.integers(0, N, size=6))
    heads = sorted({0, H // 2 - 1, H // 2, H - 1})
    q_rows = [(0, h, t) for h in heads for t in sorted(toks)]
    # key rows near the end of their group (few queries attend them, so the oracle stays fast):
    # an unshifted KV head, and a shifted one in its wrapped last group and in an interior group
    kv_rows = []
    offs = sorted({1, 2, 64, 65, 128, 129, kv_tail - 1, kv_tail})
    for off in offs:
        kv_rows.append((0, 0, G - off))                       # unshifted, group 0
        kv_rows.append((0, 0, N - off))                       # unshifted, last group
        kv_rows.append((0, Hkv - 1, (G // 2 - off) % N))      # shifted: end of the wrapped group
        kv_rows.append((0, Hkv - 1, G + G // 2 - off))        # shifted: end of group 0
    assert all(h // rep < Hkv for _, h, _ in q_rows)
    return q_rows, kv_rows


def _head_of_group_rows(w):
    """Key rows at in-group positions 0, 1, 127, 128 of group 0 of KV head 0 (unshifted) and of the
    wrapped last group of the last KV head (shifted; for the GQA shape all its query heads attend):
    almost every query of the group attends them, so their dk and dv accumulate over all query
    sub-tiles and query heads.  The oracle needs the statistics of those two units only."""
    N, G, Hkv = w.N, w.G, w.Hkv
    rows = []
    for pos in (0, 1, 127, 128):
        rows.append((0, 0, pos))
        rows.append((0, Hkv - 1, (N - G // 2 + pos) % N))
    return rows


HEAD_ROWS = {"llama2_7b_32k", "llama2_70b_32k_gqa", "llama2_7b_100k"}
GRAD_ROW_REL_L2 = 3e-2   # bound on every single sampled gradient row, beside the pooled bound


FULL = [("llama2_7b_8k", 2048), ("llama2_7b_32k", 1500), ("llama2_70b_32k_gqa", 600), ("llama2_7b_100k", 700),
        ("llama2_7b_16k", 1500), ("llama2_7b_64k", 900), ("llama2_13b_32k", 1500), ("llama2_7b_100000", 700)]


@pytest.mark.parametrize("name,kv_tail", FULL)
def test_benchmark_sizes_sampled_rows_and_properties(s2a, name, kv_tail):
    w = WORKLOADS[name]
    q, k, v, dO = make_inputs(w.B, w.N, w.H, w.Hkv, w.d, seed=0)
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    o, lse = s2a.s2a_fwd(qd, kd, vd, w.G)
    dq, dk, dv = s2a.s2a_bwd(qd, kd, vd, o, lse, dOd, w.G)
    torch.cuda.synchronize()
    rc, where = s2a.device_status()
    assert rc == 0, (rc, where)

    q_rows, kv_rows = _sample_rows(w, kv_tail)
    if name in HEAD_ROWS:
        kv_rows = kv_rows + _head_of_group_rows(w)
    o_ref, lse_ref = orc.fwd(q, k, v, w.G, rows=q_rows)
    dq_ref, dk_ref, dv_ref = orc.bwd(q, k, v, dO, w.G, q_rows=q_rows, kv_rows=kv_rows)
    qi = torch.tensor(q_rows, device=dev)
    ki = torch.tensor(kv_rows, device=dev)
    o_s = o[qi[:, 0], qi[:, 2], qi[:, 1]].double().cpu().numpy()
    lse_s = lse[qi[:, 0], qi[:, 1], qi[:, 2]].double().cpu().numpy()
    dq_s = dq[qi[:, 0], qi[:, 2], qi[:, 1]].double().cpu().numpy()
    dk_s = dk[ki[:, 0], ki[:, 2], ki[:, 1]].double().cpu().numpy()
    dv_s = dv[ki[:, 0], ki[:, 2], ki[:, 1]].double().cpu().numpy()
    assert np.abs(o_s - o_ref).max() <= O_ATOL
    assert np.abs(lse_s - lse_ref).max() <= LSE_ATOL
    assert rel_l2(dq_s, dq_ref) <= GRAD_REL_L2
    assert rel_l2(dk_s, dk_ref) <= GRAD_REL_L2
    assert rel_l2(dv_s, dv_ref) <= GRAD_REL_L2
    # no single row may be far off (rows whose exact gradient is zero, e.g. dq of the first member of a
    # group, are measured against the typical row norm)
    for got, want in ((dq_s, dq_ref), (dk_s, dk_ref), (dv_s, dv_ref)):
        row_norm = np.linalg.norm(want, axis=-1)
        floor = 0.05 * float(np.sqrt((row_norm ** 2).mean()))
        row_err = np.linalg.norm(got - want, axis=-1) / np.maximum(row_norm, floor)
        assert row_err.max() <= GRAD_ROW_REL_L2, (int(row_err.argmax()), float(row_err.max()))

    # properties that hold at any size (they touch every tile of every output)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    rep = w.H // w.Hkv
    # rows of P sum to one: sum over keys of dV equals the sum over queries of dO, per KV head
    dv_sum = dv.double().sum(dim=1)                                        # [B, Hkv, d]
    do_sum = dOd.double().view(w.B, w.N, w.Hkv, rep, w.d).sum(dim=(1, 3))  # [B, Hkv, d]
    scale_ref = dOd.double().abs().view(w.B, w.N, w.Hkv, rep, w.d).sum(dim=(1, 3))
    assert ((dv_sum - do_sum).abs() / scale_ref).max().item() < 5e-3
    # sum over (t, c) of dQ*q equals sum over (t', c) of dK*k per KV head (both are sum of dS*z)
    lhs = (dq.double() * qd.double()).view(w.B, w.N, w.Hkv, rep, w.d).sum(dim=(1, 3, 4))
    rhs = (dk.double() * kd.double()).sum(dim=(1, 3))
    mag = (dq.double() * qd.double()).abs().view(w.B, w.N, w.Hkv, rep, w.d).sum(dim=(1, 3, 4))
    assert ((lhs - rhs).abs() / mag).max().item() < 5e-3
    # the first member of every group attends only itself: o = v there
    for h in (0, w.H - 1):
        s = 0 if h < w.H // 2 else w.G // 2
        t_first = torch.tensor([(g * w.G + s) % w.N for g in range(w.N // w.G)], device=dev)
        assert torch.equal(o[0, t_first, h], vd[0, t_first, h // rep])


@pytest.mark.parametrize("B,N,G,H,Hkv,d,kw,one_head_per_pass", [
    (1, 1024, 256, 4, 4, 64, {}, False),
    (2, 2048, 512, 8, 2, 128, {}, False),
    (1, 2048, 512, 8, 2, 128, {}, True),                       # the KV heads in two passes
    (1, 2400, 600, 4, 2, 128, {}, False),                      # ragged tiles
    (1, 2400, 600, 4, 4, 64, {"leak_free": True}, True),
    (1, 2400, 600, 4, 4, 128, {"swap_wrapped": True}, False),
    (1, 4096, 1024, 6, 3, 128, {"n_unshifted": 2, "shift": 384}, False),
    (1, 4096, 4096, 2, 2, 128, {"n_unshifted": 2}, False),     # full causal attention
])
def test_spilling_backward_equals_recomputing_backward(s2a, B, N, G, H, Hkv, d, kw, one_head_per_pass):
    """With a workspace that has room for dS the dk/dv kernel spills it and dq is a plain product; with the
    minimum workspace dq recomputes the scores.  dk and dv must agree bit for bit, dq to rounding, and dq
    of the spilling path must match the oracle like any other result."""
    q, k, v, dO = make_inputs(B, N, H, Hkv, d, seed=21)
    dev = torch.device("cuda:0")
    qd, kd, vd, dOd = (x.to(dev) for x in (q, k, v, dO))
    o, lse = s2a.s2a_fwd_ex(qd, kd, vd, G, **kw)
    mn = s2a.bwd_workspace_bytes(B, N, H, Hkv, d, G)
    ref = s2a.s2a_bwd_ex(qd, kd, vd, o, lse, dOd, G, workspace=torch.empty(mn, dtype=torch.uint8, device=dev), **kw)
    full = s2a.bwd_workspace_bytes_fast(B, N, H, Hkv, d, G, 1 << 40)
    assert full > mn
    # a shift that is not a multiple of 128 adds a tile per group: leave room for it
    size = mn + 256 + (full - mn) // Hkv + 4096 if one_head_per_pass else full + (full - mn) // 2
    got = tuple(torch.full_like(x, float("nan")) for x in (qd, kd, vd))
    s2a.s2a_bwd_ex(qd, kd, vd, o, lse, dOd, G, workspace=torch.empty(size, dtype=torch.uint8, device=dev),
                   dq=got[0], dk=got[1], dv=got[2], **kw)
    torch.cuda.synchronize()
    assert s2a.device_status() == (0, 0)
    assert torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])
    assert not torch.isnan(got[0].float()).any()
    assert rel_l2(got[0].double().cpu().numpy(), ref[0].double().cpu().numpy()) <= 2e-3
    okw = dict(kw)
    dq_ref, _, _ = orc.bwd(q, k, v, dO, G, **okw)
    assert rel_l2(got[0].double().cpu().numpy(), dq_ref) <= GRAD_REL_L2
