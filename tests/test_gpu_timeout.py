"""The time-out path, seen end to end without hanging or faulting anything: a diagnostic kernel of
the library waits, with the library's own bounded wait and a short limit, on a barrier nothing
arrives on.  The wait runs out; the status must be recorded, sticky (kernels behind it do nothing,
entry points refuse on the host), readable and clearable, after which results are correct again."""
import pytest
import torch

from paper_2309_12307_b200.inputs import make_inputs

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_sticky_and_clearable():
    from paper_2309_12307_b200 import binding as s2a

    s2a.load()
    B, N, G, H, Hkv, d = 1, 1024, 256, 4, 2, 128
    q, k, v, dO = (x.cuda() for x in make_inputs(B, N, H, Hkv, d, seed=31))
    torch.cuda.synchronize()
    assert s2a.device_status() == (0, 0)
    o_ref, lse_ref = s2a.s2a_fwd(q, k, v, G)
    dq_ref, dk_ref, dv_ref = s2a.s2a_bwd(q, k, v, o_ref, lse_ref, dO, G)
    torch.cuda.synchronize()

    # A wait of 2e7 cycles (about 10 ms) that nothing ends, and a forward enqueued right behind it:
    # the host sees a clean status when it enqueues, the forward's thread blocks start after the
    # diagnostic kernel has given up, find the status word set and return without writing.
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, H, N), float("nan"), dtype=torch.float32, device="cuda")
    s2a.selftest_wait_expiry(20_000_000)
    s2a.s2a_fwd(q, k, v, G, o=o, lse=lse)
    torch.cuda.synchronize()
    assert torch.isnan(o.float()).all() and torch.isnan(lse).all()

    # now the host-visible copy is set: nothing more is enqueued until the status has been read
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_fwd(q, k, v, G, o=o, lse=lse)
    assert e.value.status == s2a.S2A_ERR_TIMEOUT
    with pytest.raises(s2a.S2AError) as e:
        s2a.s2a_bwd(q, k, v, o_ref, lse_ref, dO, G)
    assert e.value.status == s2a.S2A_ERR_TIMEOUT
    torch.cuda.synchronize()
    assert torch.isnan(o.float()).all()

    rc, where = s2a.device_status()
    assert rc == s2a.S2A_ERR_TIMEOUT and where == 901
    assert "wait" in s2a.status_string(rc)
    assert s2a.device_status() == (0, 0)          # read-and-clear

    o2, lse2 = s2a.s2a_fwd(q, k, v, G)
    dq2, dk2, dv2 = s2a.s2a_bwd(q, k, v, o2, lse2, dO, G)
    torch.cuda.synchronize()
    assert s2a.device_status() == (0, 0)
    for a, b in ((o2, o_ref), (lse2, lse_ref), (dq2, dq_ref), (dk2, dk_ref), (dv2, dv_ref)):
        assert torch.equal(a, b)


def test_selftest_rejects_limits_outside_its_range():
    from paper_2309_12307_b200 import binding as s2a

    lib = s2a.load()
    assert lib.s2a_selftest_wait_expiry(0, None) == s2a.S2A_ERR_INVALID_ARG
    assert lib.s2a_selftest_wait_expiry(3_000_000_000, None) == s2a.S2A_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert s2a.device_status() == (0, 0)
