"""The allocation-free prompt phase (`mkv_prefill_static`) against the ordinary `mkv_prefill`.

Some hosts of the library cannot let it allocate device memory: an inference server that gave
all of HBM to its own pool at start-up (a further cudaMalloc fails or fragments the pool), or
a latency-critical thread that must not run into the device-wide synchronisation of
cudaMalloc/cudaFree.  For them the library offers a prompt phase whose scratch is a fixed
16 MiB device array inside the library image.  This test calls that entry point through the C
ABI twice in a row (the second call re-uses the array with the first call's leftovers in it,
on a different prompt length) and checks, each time, that the resulting cache state and the
following decode steps equal those of the ordinary entry point.

Collected last on purpose, so that a run that stops at the first failure has already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2503_00979_b200 import binding, synth

pytestmark = pytest.mark.gpu

TOL_OUT = 2e-2      # the bf16 output tolerance of the other parity tests


def _prefill_and_decode(w, use_static, steps=6):
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    P, Rw = w.prompt_len, min(w.R, w.prompt_len)
    k, v = st.kv(np.arange(P))
    qw = st.q(np.arange(P - Rw, P))
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype)
    args = (k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
    if use_static:
        # the call must not take device memory: the CUDA runtime's free-byte count is the same before and after
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        mk.prefill_static(*args)
        mk.sync()
        assert torch.cuda.mem_get_info()[0] == free_before, "mkv_prefill_static changed the device's free memory"
    else:
        mk.prefill(*args)
    mk.sync()
    state = []
    for l in range(w.layers):
        vw = mk.view(l)
        n = vw["count"]
        state.append({name: vw[name][:, :, :n].clone() for name in ("K", "V", "pos")})
        state[-1]["ring_q"] = vw["ring_q"].clone()
        state[-1]["ring_c"] = vw["ring_c"].clone()
        state[-1]["count"] = n
    outs = []
    for i in range(steps):
        p = [P + i]
        kk, vv = st.kv(p)
        outs.append(mk.decode_step(st.q(p)[:, :, :, 0].bfloat16().contiguous(), kk[:, :, :, 0].bfloat16().contiguous(),
                                   vv[:, :, :, 0].bfloat16().contiguous()).float())
    mk.sync()
    final_pos = [torch.sort(mk.view(l)["pos"], dim=-1).values.clone() for l in range(w.layers)]
    mk.close()
    return state, torch.stack(outs), final_pos


def test_static_prefill_matches_ordinary_prefill_twice_in_a_row():
    # 12 units of (64 + 1) * 6000 floats each: more than the array holds at once, so the first call also
    # exercises the path that pushes the units through it in two batches
    base = synth.Workload("noalloc", 2, 3, 8, 2, 128, "bf16", 6000, 6, 300, 16, "sum", 31337)
    # second call: other prompt length and fusion, so the array's old contents do not line up
    for w in (base, base.replace(prompt_len=517, C=211, fusion="max", seed=4711)):
        ref_state, ref_out, ref_pos = _prefill_and_decode(w, use_static=False)
        got_state, got_out, got_pos = _prefill_and_decode(w, use_static=True)
        for a, b in zip(ref_state, got_state):
            assert a["count"] == b["count"] == w.C + w.R
            assert torch.equal(a["pos"], b["pos"])
            assert torch.equal(a["K"], b["K"]) and torch.equal(a["V"], b["V"])
            assert torch.equal(a["ring_q"], b["ring_q"])
            assert torch.allclose(a["ring_c"], b["ring_c"], rtol=0, atol=1e-5)
        assert (ref_out - got_out).abs().max().item() <= TOL_OUT
        for a, b in zip(ref_pos, got_pos):
            assert torch.equal(a, b)


def test_static_prefill_rejects_prompts_beyond_its_array():
    # (min(R,P)*G + 1) * P floats for one unit must fit 4 Mi floats: 129 * 40000 does not
    mk = binding.MorphKV(1, 1, 8, 2, 64, 2000, 32, "sum", "bf16")
    dummy = torch.zeros(8, device="cuda", dtype=torch.bfloat16)
    st = binding.mkv_prefill_static(mk.ctx, dummy, dummy, dummy, 40000)
    assert st == binding.UNSUPPORTED
    assert "4194304" in binding.mkv_last_error(mk.ctx) and "mkv_prefill" in binding.mkv_last_error(mk.ctx)
    # the context is untouched and still accepts a prompt
    k = torch.randn(1, 1, 2, 40, 64, device="cuda").bfloat16()
    qw = torch.randn(1, 1, 8, 32, 64, device="cuda").bfloat16()
    mk.prefill_static(k, k, qw)
    mk.sync()
    assert mk.view(0)["count"] == 40
    mk.close()
