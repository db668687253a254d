"""The error contract of the C ABI on a device: the status word a kernel's bounded wait writes, what
d2c_sync_status reports from it, and the argument checks that need a live context."""
import pytest
import torch

from paper_2509_23094_b200 import binding, inputs
from gpu_util import Pair

pytestmark = pytest.mark.gpu


def test_status_word_is_reported_and_sticky_until_cleared():
    wl = inputs.WORKLOADS["toy"]
    pair = Pair(wl)
    pair.gpu_step(10 ** 6, 1.0)                                     # a clean step: status stays 0
    st = pair.ctx.view("status")
    assert st.tolist() == [0, 0, 0, 0]
    # what a kernel's wait that ran out leaves behind: the code and the number of the wait
    st.copy_(torch.tensor([binding.D2C_ETIMEOUT, 32, 0, 0], dtype=torch.int32))
    with pytest.raises(binding.D2cError) as e:
        pair.ctx.sync_status()
    assert e.value.code == binding.D2C_ETIMEOUT and "site 32" in str(e.value)
    with pytest.raises(binding.D2cError):                           # sticky: still there on the next call
        pair.ctx.sync_status()
    st.zero_()
    pair.ctx.sync_status()
    g = pair.gpu_step(wl.k, wl.p)                                   # and the context is as usable as before
    assert 0 < len(g["sel"][0]) < wl.seq_len


def test_a_bounded_wait_that_runs_out_returns_and_records_the_timeout():
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    binding.d2c_op_wait_probe(status, limit_cycles=100000)          # ~50 us: nothing ever arrives on the barrier
    torch.cuda.synchronize()                                        # the kernel came back by itself
    assert status.tolist()[:2] == [binding.D2C_ETIMEOUT, 99]
    # the first error wins: a second run does not overwrite the site
    status[1] = 7
    binding.d2c_op_wait_probe(status, limit_cycles=50000)
    torch.cuda.synchronize()
    assert status.tolist()[:2] == [binding.D2C_ETIMEOUT, 7]
    # the device is fine afterwards
    x = torch.arange(8, device="cuda").sum().item()
    assert x == 28
    with pytest.raises(binding.D2cError):
        binding.d2c_op_wait_probe(status, limit_cycles=10)          # limits outside [1e3, 2e9] are refused on the host


def test_a_context_keeps_the_batch_and_length_of_its_first_step():
    wl = inputs.WORKLOADS["toy"]
    pair = Pair(wl, max_batch=2, max_seq=wl.seq_len + 64)
    pair.gpu_step(10 ** 6, 1.0)
    B, L, d = wl.batch, wl.seq_len, wl.shape.d_model
    h0 = torch.zeros(2, L, d, dtype=torch.bfloat16, device="cuda")
    mask = torch.ones(2, L, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.D2cError) as e:
        pair.ctx.step(h0, mask, 4, 0.5)                              # fits max_batch x max_seq, but is another layout
    assert e.value.code == binding.D2C_EINVAL and "first used" in str(e.value)
    with pytest.raises(binding.D2cError) as e:
        pair.ctx.step(h0[:1, : L - 8].contiguous(), mask[:1, : L - 8].contiguous(), 4, 0.5)
    assert e.value.code == binding.D2C_EINVAL
    g = pair.gpu_step(wl.k, wl.p)                                   # the original shape still works
    assert len(g["sel"][0]) > 0
