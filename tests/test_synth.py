"""The seeded input streams: determinism, slicing consistency and the stated value model."""
import numpy as np
import torch

from paper_2503_00979_b200 import synth


def test_deterministic_and_sliceable():
    w = synth.WORKLOADS["c1"].replace(layers=3, batch=2)
    st = synth.Stream(w)
    k, v = st.kv(np.arange(5, 25))
    q = st.q(np.arange(5, 25))
    assert k.shape == (3, 2, 8, 20, 128) and q.shape == (3, 2, 32, 20, 128)
    k2, v2 = synth.Stream(w).kv([7, 9], layers=[2], batch=[1], heads=[3, 5])
    assert torch.equal(k2[0, 0, 0], k[2, 1, 3, [2, 4]]) and torch.equal(v2[0, 0, 1], v[2, 1, 5, [2, 4]])
    q2 = st.q([24], layers=[1], batch=[0], kv_heads=[6])
    assert torch.equal(q2[0, 0, :, 0], q[1, 0, 24:28, 19])
    other = synth.Stream(w.replace(seed=w.seed + 1)).kv(np.arange(5, 25))[0]
    assert not torch.equal(other, k)


def test_bf16_values_are_exact_bf16():
    st = synth.Stream(synth.WORKLOADS["c1"].replace(layers=1))
    k, v = st.kv(np.arange(4))
    q = st.q(np.arange(4))
    for x in (k, v, q):
        assert torch.equal(x, x.to(torch.bfloat16).to(torch.float32))


def test_value_model_statistics():
    w = synth.WORKLOADS["c0"].replace(layers=4, batch=8, prompt_len=0)
    st = synth.Stream(w)
    k, v = st.kv(np.arange(1, 600))
    assert abs(v.mean()) < 0.01 and abs(v.std() - 1.0) < 0.01
    rms = k.pow(2).mean(-1).sqrt()                       # per-row scale: 1 or 4
    heavy = (rms > 2.5).double().mean().item()
    assert 0.015 < heavy < 0.025
    assert abs(rms[rms < 2.5].mean() - 1.0) < 0.02 and abs(rms[rms > 2.5].mean() - 4.0) < 0.1
    q = st.q(np.arange(1, 600))
    # q = 0.5 k_j + z': variance 1 + 0.25 * E[s^2] = 1 + 0.25 * (0.98 + 0.02 * 16)
    assert abs(q.var() - (1 + 0.25 * (0.98 + 0.32))) < 0.05


def test_sink_key_and_first_query():
    w = synth.WORKLOADS["c2"].replace(layers=1, batch=2)
    k, _ = synth.Stream(w).kv([0, 1])
    k_plain, _ = synth.Stream(w.replace(sink=False)).kv([0, 1])
    r = k[..., 0, :].float().norm(dim=-1) / k_plain[..., 0, :].float().norm(dim=-1)
    assert torch.allclose(r, torch.full_like(r, 8.0), rtol=1e-2)
    assert torch.equal(k[..., 1, :], k_plain[..., 1, :])
    q0 = synth.Stream(w).q([0])
    assert abs(q0.std() - 1.0) < 0.05                     # no earlier key to copy at position 0


def test_query_correlates_with_an_earlier_key():
    w = synth.WORKLOADS["c0"]
    st = synth.Stream(w)
    k, _ = st.kv(np.arange(300))
    q = st.q([299])
    logits = torch.einsum("hd,pd->hp", q[0, 0, :4, 0], k[0, 0, 0]) / 8.0
    # the matched key stands out: 0.5*|k|^2/sqrt(d) ~ 4 against a unit-ish background
    assert (logits.max(dim=1).values > 2.0).all()


def test_workload_table_matches_the_stated_configs():
    W = synth.WORKLOADS
    assert (W["c0"].units, W["c1"].units, W["c2"].units, W["c3"].units, W["c4_C512_sum"].units) == (2, 256, 8192, 2048, 1024)
    assert W["c1"].capacity == 2032 and W["c3"].capacity == 4064 and W["c4_C8192_max"].prompt_len == 8224
