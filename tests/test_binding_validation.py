"""The Python binding hands raw pointers to the C-ABI, so it must refuse, on the host and before any
call into the library, every tensor that is not what the kernels would take it for: a CPU tensor, a
wrong dtype, a non-contiguous view, or shapes that do not fit together.  No GPU is touched here."""
import pytest
import torch

from paper_2309_12307_b200 import binding as s2a


def _cpu(B=1, N=256, H=2, Hkv=2, d=64, dtype=torch.bfloat16):
    q = torch.zeros((B, N, H, d), dtype=dtype)
    k = torch.zeros((B, N, Hkv, d), dtype=dtype)
    return q, k, k.clone()


@pytest.mark.parametrize("call", ["fwd", "fwd_ex", "bwd", "bwd_ex", "noalloc", "stage"])
def test_cpu_tensors_are_refused_before_the_library_is_called(call):
    q, k, v = _cpu()
    lse = torch.zeros((1, 2, 256))
    ws = torch.zeros(4096, dtype=torch.uint8)
    with pytest.raises(ValueError, match="CUDA"):
        if call == "fwd":
            s2a.s2a_fwd(q, k, v, 128)
        elif call == "fwd_ex":
            s2a.s2a_fwd_ex(q, k, v, 128, scale=0.1)
        elif call == "bwd":
            s2a.s2a_bwd(q, k, v, q, lse, q, 128)
        elif call == "bwd_ex":
            s2a.s2a_bwd_ex(q, k, v, q, lse, q, 128)
        elif call == "noalloc":
            s2a.s2a_bwd_noalloc(q, k, v, q, lse, q, 128, q, k, v)
        else:
            s2a.s2a_bwd_stage(q, k, v, q, lse, q, 128, q, k, v, ws, 0)


def test_packed_entry_points_check_their_tensor():
    with pytest.raises(ValueError, match="CUDA"):
        s2a.s2a_fwd_packed(torch.zeros((1, 256, 3, 2, 64), dtype=torch.bfloat16), 128)
    with pytest.raises(ValueError):
        s2a.s2a_bwd_packed(torch.zeros((1, 256, 3, 2, 64), dtype=torch.float32), None, None, None, 128)


def test_shape_dtype_and_layout_rules_of_the_argument_checker():
    """The checks themselves, with the CUDA requirement switched off (it was shown above to come first)."""
    q, k, v = _cpu()
    assert s2a._dims(q, k, v, cuda=False) == (1, 256, 2, 2, 64)
    with pytest.raises(ValueError, match="dtype"):
        s2a._dims(q.float(), k, v, cuda=False)
    with pytest.raises(ValueError, match="dtype"):
        s2a._dims(q, k.half(), v, cuda=False)
    with pytest.raises(ValueError, match="k must be"):
        s2a._dims(q, k[:, :128].contiguous(), v, cuda=False)       # too few tokens
    with pytest.raises(ValueError, match="k must be"):
        s2a._dims(q, torch.zeros((1, 256, 2, 32), dtype=torch.bfloat16), v, cuda=False)   # other head dim
    with pytest.raises(ValueError, match="v must have shape"):
        s2a._dims(q, k, torch.zeros((1, 256, 1, 64), dtype=torch.bfloat16), cuda=False)   # k and v disagree
    with pytest.raises(ValueError, match="contiguous"):
        s2a._dims(q.transpose(1, 2), k, v, cuda=False)
    with pytest.raises(ValueError, match=r"\[B, N, H, d\]"):
        s2a._dims(q[0], k, v, cuda=False)
    with pytest.raises(ValueError, match="lse must have shape"):
        s2a._require(torch.zeros((1, 256, 2)), torch.float32, "lse", shape=(1, 2, 256), cuda=False)
    with pytest.raises(ValueError, match="torch.Tensor"):
        s2a._require(None, torch.float32, "lse", cuda=False)


def test_host_entry_point_checks_host_and_device_sides():
    q, k, v = _cpu()
    lse = torch.zeros((1, 2, 256))
    host_in = (q, k, v, q.clone())
    host_out = (q.clone(), lse, q.clone(), k.clone(), v.clone())
    ws = torch.zeros(4096, dtype=torch.uint8)
    with pytest.raises(ValueError, match="nine"):
        s2a.s2a_fwd_bwd_host(host_in, host_out, (q,), 128, ws)
    with pytest.raises(ValueError, match="device q"):
        s2a.s2a_fwd_bwd_host(host_in, host_out, (q, k, v, q, q, lse, q, k, v), 128, ws)   # "device" buffers on the CPU
    with pytest.raises(ValueError, match="host lse"):
        s2a.s2a_fwd_bwd_host(host_in, (q.clone(), lse.double(), q.clone(), k.clone(), v.clone()), (q,) * 9, 128, ws)
