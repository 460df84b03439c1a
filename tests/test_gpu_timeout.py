"""The bounded device-side waits: a wait that runs out must make the kernel return, be reported as
MKV_DEVICE_TIMEOUT with the code of the wait, and leave the GPU usable.  Nothing is made to fault or hang:
the limit of every wait is simply set below the latency of the first copy (mkv_params.wait_limit_cycles)."""
import numpy as np
import pytest
import torch

from paper_2503_00979_b200 import binding, synth

pytestmark = pytest.mark.gpu

W = synth.Workload("timeout", 1, 1, 8, 2, 128, "bf16", 300, 4, 200, 16, "sum", 5)


def _inputs(dev):
    st = synth.Stream(W, dev)
    k, v = st.kv(np.arange(W.prompt_len))
    qw = st.q(np.arange(W.prompt_len - W.R, W.prompt_len))
    kk, vv = st.kv([W.prompt_len])
    q = st.q([W.prompt_len])
    return (k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous(),
            q[:, :, :, 0].bfloat16().contiguous(), kk[:, :, :, 0].bfloat16().contiguous(), vv[:, :, :, 0].bfloat16().contiguous())


def test_a_wait_that_runs_out_is_reported_and_the_next_context_works():
    dev = torch.device("cuda:0")
    k, v, qw, q, kn, vn = _inputs(dev)
    # reference result from a context with the default limit
    ok = binding.MorphKV(1, 1, 8, 2, 128, W.C, W.R, W.fusion, "bf16", kernel="tc")
    ok.prefill(k, v, qw)
    want = ok.decode_step(q, kn, vn).clone()
    ok.sync()
    ok.close()

    # 50 clock ticks: no copy from global memory lands that fast, so the first wait on one gives up
    mk = binding.MorphKV(1, 1, 8, 2, 128, W.C, W.R, W.fusion, "bf16", kernel="tc", wait_limit_cycles=50)
    mk.prefill(k, v, qw)
    mk.decode_step(q, kn, vn)
    st = binding.mkv_sync(mk.ctx)
    assert st == binding.DEVICE_TIMEOUT, binding.STATUS_NAMES[st]
    msg = binding.mkv_last_error(mk.ctx)
    assert "wait code" in msg
    code = int(msg.split("wait code")[1].strip(" )"))
    assert 1 <= code <= 11, msg
    mk.close()
    torch.cuda.synchronize()

    # the device is fine: a fresh context gives the reference result bit for bit
    again = binding.MorphKV(1, 1, 8, 2, 128, W.C, W.R, W.fusion, "bf16", kernel="tc")
    again.prefill(k, v, qw)
    got = again.decode_step(q, kn, vn)
    again.sync()
    assert torch.equal(got, want)
    again.close()
