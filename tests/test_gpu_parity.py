"""Parity of the CUDA decode path (called through the C ABI) with the CPU oracle, step by step."""
import numpy as np
import pytest
import torch

from paper_2503_00979_b200 import binding, synth
from tests.parity import run_parity, run_parity_coarse, run_parity_ragged

pytestmark = pytest.mark.gpu

SMALL = synth.Workload("small", 2, 2, 8, 2, 128, "bf16", 300, 96, 200, 16, "sum", 777)


def _report(rep):
    print(f"\n[parity] kernel={rep.kernel} steps={rep.steps} unit_steps={rep.unit_steps} max_out_err={rep.max_out_err:.3e} "
          f"evictions={rep.evictions} near_tie_resyncs={rep.near_tie_resyncs} max_F_rel_err={rep.max_F_rel_err:.3e} "
          f"(F compared {rep.F_compared}) prefill_resyncs={rep.prefill_resyncs} min_rel_gap={rep.min_rel_gap:.2e}")


@pytest.mark.parametrize("seed_off", [0, 100, 200])
def test_config0_every_unit_every_step(seed_off):
    w = synth.WORKLOADS["c0"]
    rep = run_parity(w.replace(seed=w.seed + seed_off), steps=w.steps, n_units=w.units, chunk=128)
    _report(rep)
    assert rep.unit_steps == w.units * w.steps and rep.evictions > 0
    assert rep.near_tie_resyncs <= 0.01 * rep.evictions + 2


@pytest.mark.parametrize("fusion", ["sum", "max"])
@pytest.mark.parametrize("dtype,d", [("bf16", 128), ("bf16", 64), ("f32", 128), ("f32", 64)])
def test_small_shapes_simt(fusion, dtype, d):
    w = SMALL.replace(fusion=fusion, dtype=dtype, head_dim=d)
    rep = run_parity(w, steps=w.steps, n_units=8, kernel="simt")
    _report(rep)
    assert rep.evictions > 0 and rep.F_compared > 0


@pytest.mark.parametrize("G,R,C,P", [(1, 8, 100, 150), (7, 12, 90, 133), (4, 32, 2000 - 1, 2100), (16, 4, 33, 80),
                                     (2, 1, 50, 70), (4, 40, 217, 250)])
def test_group_sizes_windows_and_ragged_tails(G, R, C, P):
    # G = 1 is MHA, G = 7 the Qwen ratio; cache sizes that are no multiple of any tile
    w = SMALL.replace(layers=1, batch=2, n_q_heads=2 * G, n_kv_heads=2, R=R, C=C, prompt_len=P, steps=48, fusion="max")
    rep = run_parity(w, steps=w.steps, n_units=4, kernel="simt")
    _report(rep)
    assert rep.evictions > 0


@pytest.mark.parametrize("splits", [1, 2, 5])
def test_split_counts_give_the_same_answer(splits):
    w = SMALL.replace(layers=1, C=500, prompt_len=700, steps=40)
    rep = run_parity(w, steps=w.steps, n_units=4, kernel="simt", splits=splits)
    _report(rep)
    assert rep.evictions > 0


def test_no_eviction_regime_is_full_attention():
    # C + R >= P + S: the oracle equals plain causal attention here (pinned on the CPU side)
    w = SMALL.replace(C=400, R=16, prompt_len=100, steps=64)
    rep = run_parity(w, steps=w.steps, n_units=8)
    _report(rep)
    assert rep.evictions == 0


def test_fill_phase_then_eviction_starts():
    w = SMALL.replace(C=120, R=16, prompt_len=100, steps=80)      # fills 36 steps, then evicts
    rep = run_parity(w, steps=w.steps, n_units=8)
    _report(rep)
    assert rep.evictions == 8 * (80 - 36)


def test_prompt_shorter_than_the_window():
    w = SMALL.replace(C=20, R=16, prompt_len=5, steps=60, layers=1)
    rep = run_parity(w, steps=w.steps, n_units=4)
    _report(rep)
    assert rep.evictions > 0


def test_single_token_prompt():
    w = SMALL.replace(C=6, R=3, prompt_len=1, steps=30, layers=1)
    rep = run_parity(w, steps=w.steps, n_units=4)
    _report(rep)


def test_attention_sink_workload():
    w = synth.WORKLOADS["c2"].replace(layers=1, batch=2, prompt_len=600, C=256, steps=64)
    rep = run_parity(w, steps=w.steps, n_units=8)
    _report(rep)
    assert rep.evictions > 0


def test_decode_steps_call_and_host_call():
    w = SMALL.replace(layers=1, steps=32)
    rep = run_parity(w, steps=w.steps, n_units=4, use_steps_call=True)
    _report(rep)
    rep = run_parity(w, steps=w.steps, n_units=4, host_call_every=3)
    _report(rep)
    assert rep.evictions > 0


def test_state_order_and_argument_errors():
    mk = binding.MorphKV(1, 1, 8, 2, 64, 16, 4, "sum", "f32")
    q = torch.zeros(1, 1, 8, 64, device="cuda")
    kv = torch.zeros(1, 1, 2, 64, device="cuda")
    assert binding.mkv_decode_step(mk.ctx, q, kv, kv, q) == binding.BAD_STATE
    assert "prefill" in binding.mkv_last_error(mk.ctx)
    assert binding.mkv_prefill(mk.ctx, None, None, None, 4) == binding.INVALID_ARG
    k = torch.randn(1, 1, 2, 5, 64, device="cuda")
    qw = torch.randn(1, 1, 8, 4, 64, device="cuda")
    assert binding.mkv_prefill(mk.ctx, k, k, qw, 0) == binding.INVALID_ARG
    mk.prefill(k, k, qw)
    assert binding.mkv_prefill(mk.ctx, k, k, qw, 5) == binding.BAD_STATE
    assert binding.mkv_decode_step(mk.ctx, q, kv, None, q) == binding.INVALID_ARG
    st, v = binding.mkv_cache_view(mk.ctx, 3)
    assert st == binding.INVALID_ARG
    mk.decode_step(q, kv, kv)
    mk.sync()
    assert mk.view(0)["count"] == 6 and mk.view(0)["next_pos"] == 6 and mk.launch_count > 0
    mk.close()


def test_workspace_too_small_is_oom():
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 1, 1, 8, 2, 64, 16, 4
    buf = torch.empty(4096, dtype=torch.uint8, device="cuda")
    p.workspace, p.workspace_bytes = (buf.data_ptr() + 255) & ~255, 1024
    st, h = binding.mkv_create_ex(p)
    assert st == binding.OOM and h is None
    p.workspace = ((buf.data_ptr() + 255) & ~255) + 8       # misaligned
    st, h = binding.mkv_create_ex(p)
    assert st == binding.INVALID_ARG


def test_slot_permutation_does_not_change_results():
    # physical slot order is free: swapping two cached rows (K, V, pos together) changes nothing
    w = SMALL.replace(layers=1, batch=1, steps=8)
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    k, v = st.kv(np.arange(w.prompt_len))
    qw = st.q(np.arange(w.prompt_len - w.R, w.prompt_len))
    outs = []
    for swap in (False, True):
        mk = binding.MorphKV(1, 1, 8, 2, 128, w.C, w.R, w.fusion, "bf16")
        mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
        mk.sync()
        if swap:
            vw = mk.view(0)
            perm = torch.randperm(vw["count"], device=dev)
            for name in ("K", "V", "pos"):
                t = vw[name]
                t[:, :, :vw["count"]] = t[:, :, :vw["count"]][:, :, perm].clone()
        res = []
        for i in range(w.steps):
            p = [w.prompt_len + i]
            kk, vv = st.kv(p)
            o = mk.decode_step(st.q(p)[:, :, :, 0].bfloat16().contiguous(), kk[:, :, :, 0].bfloat16().contiguous(),
                               vv[:, :, :, 0].bfloat16().contiguous())
            res.append(o.float())
        mk.sync()
        vw = mk.view(0)
        outs.append((torch.stack(res), torch.sort(vw["pos"][0, :, :vw["count"]], dim=-1).values.clone()))
        mk.close()
    assert torch.equal(outs[0][1], outs[1][1])
    assert (outs[0][0] - outs[1][0]).abs().max() < 2e-2


# ---- tensor-core kernel (bf16, d = 128) ----------------------------------------------------
def test_tc_smallest_case_first():
    w = SMALL.replace(layers=1, batch=1, steps=24)
    rep = run_parity(w, steps=w.steps, n_units=2, kernel="tc")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0


def test_auto_picks_the_tensor_core_kernel_for_bf16_d128():
    mk = binding.MorphKV(1, 1, 8, 2, 128, 64, 16, "sum", "bf16")
    assert mk.kernel_name == "tc"
    mk.close()
    mk = binding.MorphKV(1, 1, 8, 2, 64, 64, 16, "sum", "bf16")
    assert mk.kernel_name == "simt"
    mk.close()
    mk = binding.MorphKV(1, 1, 14, 2, 128, 64, 16, "sum", "bf16")      # G = 7: group padded to 8 on the tensor cores
    assert mk.kernel_name == "tc" and mk.view(0)["ring_c"].shape[-1] == 8
    mk.close()
    p = binding.mkv_default_params()
    mk = binding.MorphKV(1, 1, 14, 2, 128, 64, 40, "sum", "bf16")      # 40 * 8 = 320 ring rows: two chunks
    assert mk.kernel_name == "tc"
    mk.close()
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 1, 1, 14, 2, 128, 64, 300    # 2400 rows: more than 8 chunks
    p.kernel = binding.KERNEL["tc"]
    st, h = binding.mkv_create_ex(p)
    assert st == binding.UNSUPPORTED and h is None
    mk = binding.MorphKV(1, 1, 14, 2, 128, 64, 300, "sum", "bf16")
    assert mk.kernel_name == "simt"
    mk.close()


@pytest.mark.parametrize("fusion", ["sum", "max"])
@pytest.mark.parametrize("G,R", [(1, 32), (2, 24), (4, 32), (4, 30), (8, 16), (16, 9), (4, 64), (7, 30), (3, 20), (6, 12)])
def test_tc_groups_windows_and_fusions(fusion, G, R):
    # R*G = 120 and 144 are padded to a multiple of 32; R*G = 256 fills both accumulator buffers; G = 7 (the 28/4 head
    # ratio of the LongWriter table's Qwen row), 3 and 6 run with the group padded to the next power of two
    w = SMALL.replace(layers=1, batch=2, n_q_heads=2 * G, n_kv_heads=2, R=R, C=301, prompt_len=411, steps=40,
                      fusion=fusion)
    rep = run_parity(w, steps=w.steps, n_units=4, kernel="tc")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0 and rep.F_compared > 0


@pytest.mark.parametrize("ipu", [1, 2, 3, 7])
def test_tc_item_counts_give_the_same_answer(ipu):
    w = SMALL.replace(layers=1, C=1500, R=32, prompt_len=1700, steps=36, fusion="max")     # 12 tiles, ragged tail
    rep = run_parity(w, steps=w.steps, n_units=4, kernel="tc", splits=ipu)
    _report(rep)
    assert rep.evictions > 0


@pytest.mark.parametrize("pinned", [True, False])
def test_tc_host_buffers_pinned_in_place_and_pageable_staged(pinned):
    # pinned host buffers are read and written in place by the kernel, pageable ones go through staging copies
    w = SMALL.replace(layers=2, C=300, R=32, prompt_len=400, steps=24)
    rep = run_parity(w, steps=w.steps, n_units=4, kernel="tc", host_call_every=2, host_pinned=pinned)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0


def test_tc_fill_phase_warmup_and_single_tile():
    rep = run_parity(SMALL.replace(C=120, R=16, prompt_len=100, steps=80), steps=80, n_units=8, kernel="tc")
    _report(rep)
    assert rep.evictions == 8 * (80 - 36)
    rep = run_parity(SMALL.replace(C=20, R=16, prompt_len=5, steps=60, layers=1), steps=60, n_units=4, kernel="tc")
    _report(rep)
    assert rep.evictions > 0
    rep = run_parity(SMALL.replace(C=300, R=16, prompt_len=120, steps=190, layers=1), steps=190, n_units=4, kernel="tc")
    _report(rep)       # crosses from one tile to three while filling
    assert rep.evictions == 0


def test_tc_llama_shape_two_layers():
    w = synth.WORKLOADS["c1"].replace(layers=2, steps=96)
    rep = run_parity(w, steps=w.steps, n_units=8, kernel="tc")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions == 8 * 96


def test_tc_stress_shape_window_64():
    w = synth.WORKLOADS["c3"].replace(layers=1, batch=2, prompt_len=4100, steps=48)    # starts full: C=4000, R=64
    rep = run_parity(w, steps=w.steps, n_units=6, kernel="tc")
    _report(rep)
    assert rep.evictions > 0


def test_full_size_config1_fill_phase_launched_back_to_back():
    # a prompt shorter than C + R: 96 steps that append without evicting, all launches enqueued without a
    # synchronisation in between (the regime in which a kernel variant that skipped the scoring used to fault)
    w = synth.WORKLOADS["c1"].replace(prompt_len=1500)
    rep = run_parity(w, steps=96, n_units=6, kernel="auto", chunk=48, use_steps_call=True)
    _report(rep)
    assert rep.kernel == "tc" and rep.unit_steps == 6 * 96


def test_full_size_config1_coarse_grained_launched_back_to_back():
    # T = 8 at the benchmark's size, 64 steps enqueued at once: the fill must cycle C+R .. C+R+T-1 and every
    # unit must end with a dense prefix of distinct positions that contains the whole recent window
    w = synth.WORKLOADS["c1"]
    T, steps = 8, 64
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    P = w.prompt_len
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype,
                         evict_interval=T)
    ks, vs, qs = [], [], []
    for l in range(w.layers):
        k, v = st.kv(np.arange(P), [l])
        ks.append(k.bfloat16()); vs.append(v.bfloat16()); qs.append(st.q(np.arange(P - w.R, P), [l]).bfloat16())
    mk.prefill(torch.cat(ks).contiguous(), torch.cat(vs).contiguous(), torch.cat(qs).contiguous())
    pos = np.arange(P, P + steps)
    kk, vv = st.kv(pos)
    q = st.q(pos).permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    kn = kk.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    vn = vv.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    out = torch.empty_like(q)
    mk.decode_steps(q, kn, vn, out)
    mk.sync()
    assert torch.isfinite(out.float()).all()
    view = mk.view(w.layers - 1)
    assert view["count"] == w.C + w.R                      # 64 = 8 policy steps: just compacted
    p = view["pos"][:, :, :view["count"]].cpu().numpy()
    for b in range(p.shape[0]):
        for h in range(p.shape[1]):
            row = p[b, h]
            assert len(set(row.tolist())) == len(row) and row.min() >= 0
            assert set(range(P + steps - w.R, P + steps)) <= set(row.tolist())
    assert (view["pos"][:, :, view["count"]:].cpu().numpy() == -1).all()
    mk.close()


@pytest.mark.parametrize("kernel", ["auto", "simt"])
def test_longgenbench_shape_window_200(kernel):
    # R = 200 with a 4K budget (the LongGenBench setting): R*G = 800 ring rows.  The tensor-core kernel cuts the ring
    # into four chunks of 56 slots; the prompt length makes the new query's slot cross from chunk 0 to chunk 1.
    w = synth.Workload("r200", 1, 1, 8, 2, 128, "bf16", 4250, 24, 3896, 200, "sum", 31)
    rep = run_parity(w, steps=w.steps, n_units=2, kernel=kernel, check_F_every=8)
    _report(rep)
    assert rep.kernel == ("tc" if kernel == "auto" else "simt") and rep.evictions == 2 * 24


@pytest.mark.parametrize("q_heads,kv_heads,R,C,P,fusion", [(14, 2, 40, 300, 420, "max"),     # group 7 -> 8, two chunks of 20 slots
                                                           (8, 2, 65, 300, 300, "sum"),      # 260 rows: chunks of 160; starts in the fill phase
                                                           (32, 2, 33, 200, 300, "max"),     # group 16, three chunks
                                                           (2, 2, 300, 700, 1100, "sum")])   # MHA, window 300: two chunks
def test_windows_of_more_than_256_ring_rows_on_the_tensor_cores(q_heads, kv_heads, R, C, P, fusion):
    # many small units (several work items per CTA) as well as units shared by several CTAs; prompts shorter than
    # C + R start in the fill phase, where only the chunk with the new query's slot is walked
    w = synth.Workload("wide", 2, 2, q_heads, kv_heads, 128, "bf16", P, 2 * R + 9, C, R, fusion, 77 + R)
    rep = run_parity(w, steps=w.steps, n_units=8, kernel="auto", check_F_every=5)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0


def test_wide_window_with_a_prompt_shorter_than_the_window():
    # 150 prompt tokens under a window of 200 (600 window rows: the prompt phase takes them in three pieces and has
    # no candidates to score); the cache fills for 150 steps, then every step evicts while rows of the prompt are
    # still inside the window, so the fused scores depend on the normalisers the prompt phase wrote
    w = synth.Workload("wide_short_prompt", 1, 2, 8, 2, 128, "bf16", 150, 170, 100, 200, "sum", 2024)
    rep = run_parity(w, steps=w.steps, n_units=4, kernel="auto", check_F_every=5)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions == 4 * 20 and rep.F_compared > 0


def test_wide_window_with_per_layer_calls_and_current_normalisation():
    w = synth.Workload("wide_layer", 3, 1, 8, 2, 128, "bf16", 500, 90, 400, 70, "sum", 5)
    rep = run_parity(w, steps=w.steps, n_units=6, kernel="auto", per_layer=1)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0
    rep = run_parity(w, steps=w.steps, n_units=6, kernel="auto", norm="current")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0


def test_wide_window_with_coarse_grained_eviction():
    w = synth.Workload("wide_coarse", 1, 2, 8, 2, 128, "bf16", 700, 40, 500, 80, "max", 4243)
    rep = run_parity_coarse(w, 4, steps=5 * 4 + 2, n_units=4, kernel="tc")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions == 4 * 5 * 4


# ---- coarse-grained eviction: the policy runs every T-th step and drops several tokens at once
@pytest.mark.parametrize("kernel,dtype,d", [("simt", "f32", 64), ("simt", "bf16", 128), ("tc", "bf16", 128)])
@pytest.mark.parametrize("T,fusion", [(8, "sum"), (3, "max")])
def test_coarse_grained_eviction(kernel, dtype, d, T, fusion):
    w = synth.Workload("coarse", 1, 2, 8, 2, d, dtype, 260, 40, 150, 16, fusion, 4242)
    rep = run_parity_coarse(w, T, steps=5 * T + 2, n_units=4, kernel=kernel)
    _report(rep)
    assert rep.kernel == kernel
    assert rep.evictions == 4 * 5 * T               # T tokens per policy step and unit, five policy steps
    assert rep.F_compared == w.C + w.R + T - 1      # the fill peaks one step before the policy runs


def test_coarse_grained_eviction_while_the_cache_fills():
    # prompt shorter than C + R: nothing is dropped until the older tokens exceed C on a policy step
    w = synth.Workload("coarse_fill", 1, 1, 8, 2, 128, "bf16", 100, 64, 120, 16, "sum", 99)
    rep = run_parity_coarse(w, 4, steps=64, n_units=2, kernel="tc")
    _report(rep)
    assert rep.evictions > 0


# ---- the benchmark's own sizes: every unit runs on the device, a seeded sample (first and last
# layer / batch row included) is followed by the oracle step by step
def test_full_size_config1_sampled_units():
    w = synth.WORKLOADS["c1"]
    rep = run_parity(w, steps=64, n_units=8, kernel="auto", check_F_every=32)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions >= 7 * 64


def test_full_size_config2_sampled_units():
    w = synth.WORKLOADS["c2"]
    rep = run_parity(w, steps=48, n_units=8, kernel="auto", check_F_every=24)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions >= 7 * 48


def test_full_size_config3_sampled_units_full_cache():
    # config 3 fills its cache over thousands of steps; start it full so the sample sees evictions
    w = synth.WORKLOADS["c3"].replace(prompt_len=4100)
    rep = run_parity(w, steps=24, n_units=6, kernel="auto", check_F_every=12)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions >= 5 * 24


@pytest.mark.parametrize("name", [f"c4_C{C}_{f}" for C in (512, 1024, 2048, 4096, 8192) for f in ("sum", "max")])
def test_full_size_config4_sampled_units(name):
    # every point of the capacity sweep, both fusions
    w = synth.WORKLOADS[name]
    steps = 48 if w.C <= 512 else 32 if w.C <= 2048 else 16
    rep = run_parity(w, steps=steps, n_units=6, kernel="auto", check_F_every=8)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions >= 5 * steps


# ---- the configurations over their whole length: every generated step of a seeded sample of units (first and
# last layer / batch row included) is followed by the oracle; all other units run on the device beside them
def test_full_length_config1_every_generated_step():
    w = synth.WORKLOADS["c1"]
    rep = run_parity(w, steps=w.steps, n_units=8, chunk=256, check_F_every=1024)
    _report(rep)
    assert rep.kernel == "tc" and rep.steps == 8192 and rep.units == 8
    assert rep.evictions == 8 * 8192 and rep.near_tie_resyncs <= 0.002 * rep.evictions + 2


def test_full_length_config2_every_generated_step():
    w = synth.WORKLOADS["c2"]
    rep = run_parity(w, steps=w.steps, n_units=8, chunk=64, check_F_every=512)
    _report(rep)
    assert rep.kernel == "tc" and rep.steps == 4096 and rep.units == 8
    assert rep.evictions == 8 * 4096 and rep.near_tie_resyncs <= 0.002 * rep.evictions + 2


@pytest.mark.parametrize("name", [f"c4_C{C}_{f}" for C in (512, 1024, 2048, 4096, 8192) for f in ("sum", "max")])
def test_full_length_config4_every_generated_step(name):
    # every point of the capacity sweep over all of its 1024 steps
    w = synth.WORKLOADS[name]
    rep = run_parity(w, steps=w.steps, n_units=4, chunk=128, check_F_every=256)
    _report(rep)
    assert rep.kernel == "tc" and rep.steps == 1024 and rep.units == 4
    assert rep.evictions == 4 * 1024 and rep.near_tie_resyncs <= 0.002 * rep.evictions + 2


def test_config3_from_its_real_prompt_through_the_fill_into_eviction():
    # 512-token prompt: 3552 steps that only append, then the cache is full (C + R = 4064) and every step evicts
    w = synth.WORKLOADS["c3"]
    fill = w.C + w.R - w.prompt_len
    steps = fill + 544
    rep = run_parity(w, steps=steps, n_units=4, chunk=128, check_F_every=128)
    _report(rep)
    assert rep.kernel == "tc" and rep.units == 4
    assert rep.evictions == 4 * 544 and rep.F_compared > 0


def test_config1_all_units_prompt_phase_and_first_steps_against_the_oracle():
    # every one of the 256 units: retained set after the prompt phase (near-tie rule), K/V rows bit for bit, then
    # 16 decode steps with outputs and evictions compared
    w = synth.WORKLOADS["c1"]
    rep = run_parity(w, steps=16, n_units=w.units, chunk=16, check_F_every=16)
    _report(rep)
    assert rep.units == 256 and rep.unit_steps == 256 * 16 and rep.evictions == 256 * 16
    assert rep.prefill_resyncs <= 2


# ---- long prompts into a 2K cache (the long-context setting): the prompt phase on the tensor cores
@pytest.mark.parametrize("name,layers,n_units", [("prefill_P6144", 4, 8), ("prefill_P32768", 1, 3),
                                                 ("prefill_w200_P6144", 2, 4)])      # window of 200: four pieces
def test_long_prompt_selection_against_the_oracle(name, layers, n_units):
    # retained set of every checked unit against the oracle's one-shot Algorithm 1 (near-tie rule), kept K/V rows
    # bit for bit, then a few decode steps whose outputs depend on the window rows' normalisers
    w = synth.WORKLOADS[name].replace(layers=layers)
    rep = run_parity(w, steps=8, n_units=n_units, chunk=8, check_F_every=8)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions == rep.units * 8 and rep.prefill_resyncs <= 1


@pytest.mark.parametrize("q_heads,kv_heads,R,pieces,profile", [(8, 2, 200, 4, "recompute"), (14, 2, 40, 2, "recompute"),
                                                                (8, 2, 32, 1, "recompute"), (8, 2, 700, 11, "stored")])
def test_prompt_phase_of_a_wide_window_scores_on_the_tensor_cores(q_heads, kv_heads, R, pieces, profile):
    # a window of more than 256 rows R * G' is scored in pieces of 256 / G' window slots, one pair of tensor-core
    # passes per piece: the call then launches arena set-up, 2 x pieces scoring passes, the selection, the gather,
    # the ring copy and the state kernel (the CUDA-core scoring path would launch two or three scoring kernels instead);
    # that the pieces' scores fuse to the oracle's is what the wide-window parity tests above check
    w = synth.Workload("wide_prompt", 1, 1, q_heads, kv_heads, 128, "bf16", 900, 4, 500, R, "sum", 3)
    st = synth.Stream(w, torch.device("cuda:0"))
    k, v = st.kv(np.arange(w.prompt_len))
    qw = st.q(np.arange(w.prompt_len - R, w.prompt_len))
    mk = binding.MorphKV(1, 1, q_heads, kv_heads, 128, w.C, R, w.fusion, "bf16", profile=profile)
    assert mk.kernel_name == "tc"
    n0 = mk.launch_count
    mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
    # (a window of 700 keeps the whole 900-token prompt: the position kernel stands in for the selection; the stored
    # profile adds the launch that fills its table)
    assert mk.launch_count - n0 == 1 + 2 * pieces + 1 + 2 + 1 + (1 if profile == "stored" else 0)
    mk.close()


def test_reset_lets_a_context_take_the_next_prompt():
    w = SMALL.replace(layers=1, batch=1)
    dev = torch.device("cuda:0")
    mk = binding.MorphKV(1, 1, 8, 2, 128, w.C, w.R, w.fusion, "bf16")
    got = []
    for seed in (1, 2, 1):
        st = synth.Stream(w.replace(seed=seed), dev)
        k, v = st.kv(np.arange(w.prompt_len))
        qw = st.q(np.arange(w.prompt_len - w.R, w.prompt_len))
        if got:
            assert binding.mkv_prefill(mk.ctx, k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous(),
                                       w.prompt_len) == binding.BAD_STATE
            mk.reset()
        mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
        kk, vv = st.kv([w.prompt_len])
        o = mk.decode_step(st.q([w.prompt_len])[:, :, :, 0].bfloat16().contiguous(), kk[:, :, :, 0].bfloat16().contiguous(),
                           vv[:, :, :, 0].bfloat16().contiguous())
        mk.sync()
        got.append((o.clone(), torch.sort(mk.view(0)["pos"], dim=-1).values.clone()))
    assert torch.equal(got[0][0], got[2][0]) and torch.equal(got[0][1], got[2][1])
    assert not torch.equal(got[0][0], got[1][0])
    mk.close()


# ---- the other reading of Eq. 4: window rows renormalised over the tokens still cached
@pytest.mark.parametrize("kernel,dtype,d", [("tc", "bf16", 128), ("simt", "f32", 64), ("simt", "bf16", 64)])
@pytest.mark.parametrize("fusion", ["sum", "max"])
def test_current_normalisation_against_the_oracle(kernel, dtype, d, fusion):
    w = SMALL.replace(layers=1, batch=2, head_dim=d, dtype=dtype, C=300, R=16, prompt_len=420, steps=64, fusion=fusion)
    rep = run_parity(w, steps=w.steps, n_units=4, kernel=kernel, norm="current")
    _report(rep)
    assert rep.kernel == kernel and rep.evictions == 4 * 64 and rep.F_compared > 0


def test_current_normalisation_differs_from_frozen_and_rejects_coarse_eviction():
    w = SMALL.replace(layers=1, batch=1, C=200, R=16, prompt_len=300, steps=48, fusion="sum")
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    k, v = st.kv(np.arange(w.prompt_len))
    qw = st.q(np.arange(w.prompt_len - w.R, w.prompt_len))
    pos = np.arange(w.prompt_len, w.prompt_len + w.steps)
    kk, vv = st.kv(pos)
    qn = st.q(pos).permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    kn = kk.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    vn = vv.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    cs = []
    for norm in ("frozen", "current"):
        mk = binding.MorphKV(1, 1, 8, 2, 128, w.C, w.R, w.fusion, "bf16", norm=norm)
        mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
        mk.decode_steps(qn, kn, vn)
        mk.sync()
        cs.append(mk.view(0)["ring_c"].clone())
        mk.close()
    # evicted mass leaves the rows' normalisers (and the two policies soon keep different tokens)
    assert not torch.allclose(cs[0], cs[1], rtol=0, atol=1e-3) and cs[1].mean() < cs[0].mean()
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 1, 1, 8, 2, 128, 64, 16
    p.norm_mode, p.evict_interval = binding.NORM["current"], 4
    st_, h = binding.mkv_create_ex(p)
    assert st_ == binding.UNSUPPORTED and h is None


# ---- per-layer entry (a model that runs its layers one after the other) and the layer-aware variant
@pytest.mark.parametrize("kernel,dtype,d", [("tc", "bf16", 128), ("simt", "f32", 64)])
@pytest.mark.parametrize("mode", [1, 2])
def test_per_layer_calls_against_the_oracle(kernel, dtype, d, mode):
    # mode 1: every step layer by layer; mode 2: whole-stack and per-layer steps alternate in one context
    w = SMALL.replace(layers=3, batch=2, head_dim=d, dtype=dtype, C=600, R=16, prompt_len=700, steps=40, fusion="max")
    rep = run_parity(w, steps=w.steps, n_units=6, kernel=kernel, per_layer=mode)
    _report(rep)
    assert rep.kernel == kernel and rep.evictions == 6 * 40 and rep.F_compared > 0


def test_per_layer_calls_give_the_whole_stack_results():
    # config 1's shape on four layers: a step made of per-layer calls against the same step as one call.  The two
    # cut a unit's tiles into different ranges, so outputs agree to rounding, evictions exactly.
    w = synth.WORKLOADS["c1"].replace(layers=4, steps=24)
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    P = w.prompt_len
    k, v = st.kv(np.arange(P))
    qw = st.q(np.arange(P - w.R, P))
    pos = np.arange(P, P + w.steps)
    kk, vv = st.kv(pos)
    qn = st.q(pos).permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    kn = kk.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    vn = vv.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    res = []
    for per_layer in (False, True):
        mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype)
        mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
        out = torch.empty_like(qn)
        ev = []
        for i in range(w.steps):
            if per_layer:
                for l in range(w.layers):
                    mk.decode_step_layer(l, qn[i, l], kn[i, l], vn[i, l], out[i, l])
            else:
                mk.decode_step(qn[i], kn[i], vn[i], out[i])
            ev.append(torch.stack([mk.view(l)["evicted_pos"].clone() for l in range(w.layers)]))
        mk.sync()
        assert mk.view(0)["next_pos"] == P + w.steps
        res.append((out.float(), torch.stack(ev), torch.stack([torch.sort(mk.view(l)["pos"], dim=-1).values for l in range(w.layers)])))
        mk.close()
    assert torch.equal(res[0][1], res[1][1]) and torch.equal(res[0][2], res[1][2])
    assert ((res[0][0] - res[1][0]).abs() <= 2 ** -7 * res[0][0].abs() + 1e-3).all()


def test_per_layer_calls_must_come_in_order():
    w = SMALL.replace(layers=3, batch=1, steps=1)
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    k, v = st.kv(np.arange(w.prompt_len))
    qw = st.q(np.arange(w.prompt_len - w.R, w.prompt_len))
    mk = binding.MorphKV(3, 1, 8, 2, 128, w.C, w.R, w.fusion, "bf16")
    mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
    q = torch.zeros(1, 8, 128, dtype=torch.bfloat16, device=dev)
    kv = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device=dev)
    qa = torch.zeros(3, 1, 8, 128, dtype=torch.bfloat16, device=dev)
    kva = torch.zeros(3, 1, 2, 128, dtype=torch.bfloat16, device=dev)
    assert binding.mkv_decode_step_layer(mk.ctx, 1, q, kv, kv, q) == binding.BAD_STATE          # layer 0 comes first
    assert binding.mkv_decode_step_layer(mk.ctx, 3, q, kv, kv, q) == binding.INVALID_ARG
    assert binding.mkv_decode_step_layer(mk.ctx, 0, q, kv, kv, q) == binding.OK
    assert binding.mkv_decode_step(mk.ctx, qa, kva, kva, qa) == binding.BAD_STATE                # the step has layers left
    assert binding.mkv_decode_step_layer(mk.ctx, 0, q, kv, kv, q) == binding.BAD_STATE
    assert binding.mkv_decode_step_layer(mk.ctx, 1, q, kv, kv, q) == binding.OK
    assert binding.mkv_decode_step_layer(mk.ctx, 2, q, kv, kv, q) == binding.OK
    mk.sync()
    assert mk.view(0)["next_pos"] == w.prompt_len + 1 and mk.view(2)["count"] == mk.view(0)["count"]
    assert binding.mkv_decode_step(mk.ctx, qa, kva, kva, qa) == binding.OK
    mk.sync()
    mk.close()


@pytest.mark.parametrize("per_layer", [0, 1])
def test_layer_aware_variant_first_layers_keep_every_token(per_layer):
    # MorphKV off for the first two of four layers: their units equal full attention (an oracle unit whose capacity
    # is never reached), the others evict as usual
    w = SMALL.replace(layers=4, batch=2, C=250, R=16, prompt_len=320, steps=48, fusion="sum")
    rep = run_parity(w, steps=w.steps, units=[(0, 0, 0), (1, 1, 1), (2, 0, 1), (3, 1, 0)], per_layer=per_layer,
                     full_layers=2, max_tokens=400)
    _report(rep)
    assert rep.evictions == 2 * 48            # only the two units of the MorphKV layers evict


def test_tc_matches_cuda_core_kernel_on_device():
    # the two kernels share only the per-unit epilogue; their outputs must agree closely
    w = SMALL.replace(layers=1, batch=2, C=700, R=32, prompt_len=900, steps=12, fusion="max")
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    k, v = st.kv(np.arange(w.prompt_len))
    qw = st.q(np.arange(w.prompt_len - w.R, w.prompt_len))
    res = {}
    for kern in ("simt", "tc"):
        mk = binding.MorphKV(1, 2, 8, 2, 128, w.C, w.R, w.fusion, "bf16", kernel=kern)
        mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
        outs, ev = [], []
        for i in range(w.steps):
            p = [w.prompt_len + i]
            kk, vv = st.kv(p)
            outs.append(mk.decode_step(st.q(p)[:, :, :, 0].bfloat16().contiguous(), kk[:, :, :, 0].bfloat16().contiguous(),
                                       vv[:, :, :, 0].bfloat16().contiguous()).float())
            ev.append(mk.view(0)["evicted_pos"].clone())
        mk.sync()
        res[kern] = (torch.stack(outs), torch.stack(ev), mk.view(0)["ring_c"].clone())
        mk.close()
    assert torch.equal(res["simt"][1], res["tc"][1])
    assert (res["simt"][0] - res["tc"][0]).abs().max() <= 2 ** -6       # one bf16 ulp at |o| < 4
    assert torch.allclose(res["simt"][2], res["tc"][2], rtol=0, atol=2e-4)


@pytest.mark.parametrize("name,prompt_len,steps,reps", [("c1", 4096, 48, 5), ("c1", 1500, 96, 5), ("c2", 2048, 10, 2),
                                                        ("c3", 4100, 8, 2)])
def test_full_size_every_unit_matches_cuda_core_kernel(name, prompt_len, steps, reps):
    # Every unit of a benchmark configuration on every step, launches enqueued back to back, repeated: the
    # tensor-core kernel against the CUDA-core kernel (the oracle follows a handful of units only).  This is the
    # test that shows a V stage being refilled under its last reads: on config 1, one 16-column block of the output
    # of a unit whose tiles end a CTA's range came out wrong about ten times per repetition before the readers
    # fenced their reads against the refill.  Configs 2 and 3 run fewer steps: their CUDA-core reference takes
    # tens of milliseconds per step.
    w = synth.WORKLOADS[name].replace(prompt_len=prompt_len)
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    P, Rw = prompt_len, min(w.R, prompt_len)
    ks, vs, qs = [], [], []
    for l in range(w.layers):
        k, v = st.kv(np.arange(P), [l])
        ks.append(k.bfloat16()); vs.append(v.bfloat16()); qs.append(st.q(np.arange(P - Rw, P), [l]).bfloat16())
    kp, vp, qp = torch.cat(ks).contiguous(), torch.cat(vs).contiguous(), torch.cat(qs).contiguous()
    del ks, vs, qs
    pos = np.arange(P, P + steps)
    kk, vv = st.kv(pos)
    qn = st.q(pos).permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    kn = kk.permute(3, 0, 1, 2, 4).bfloat16().contiguous()
    vn = vv.permute(3, 0, 1, 2, 4).bfloat16().contiguous()

    def run(kernel):
        mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.C, w.R, w.fusion, w.dtype,
                             kernel=kernel)
        assert mk.kernel_name == kernel
        mk.prefill(kp, vp, qp)
        out = mk.decode_steps(qn, kn, vn)
        mk.sync()
        res = out.float()
        mk.close()
        return res

    ref = run("simt")
    for _ in range(reps):
        # both outputs are rounded to bf16: allow the absolute tolerance of the parity tests plus one bf16 ulp of
        # the value (config 2's attention sink gives outputs beyond 4, where one ulp is 2^-5)
        excess = float(((run("tc") - ref).abs() - 2e-2 - ref.abs() * 2 ** -7).max())
        assert excess <= 0, f"tensor-core and CUDA-core outputs differ by {excess:.3e} more than the tolerance"


@pytest.mark.parametrize("ipu", [0, 1])
def test_tc_runs_are_bitwise_reproducible(ipu):
    # static work assignment and fixed merge order: two runs on the same inputs agree bit for bit
    # (this caught a warp-divergence bug in front of ldmatrix / mma.sync that tolerances had hidden)
    w = SMALL.replace(layers=1, batch=2, C=1500, R=32, prompt_len=1700, steps=40, fusion="max")
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    k, v = st.kv(np.arange(w.prompt_len))
    qw = st.q(np.arange(w.prompt_len - w.R, w.prompt_len))
    pos = np.arange(w.prompt_len, w.prompt_len + w.steps)
    kk, vv = st.kv(pos)
    qq = st.q(pos)
    runs = []
    for _ in range(3):
        mk = binding.MorphKV(1, 2, 8, 2, 128, w.C, w.R, w.fusion, "bf16", kernel="tc", splits=ipu)
        mk.prefill(k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous())
        outs = [mk.decode_step(qq[:, :, :, i].bfloat16().contiguous(), kk[:, :, :, i].bfloat16().contiguous(),
                               vv[:, :, :, i].bfloat16().contiguous()).clone() for i in range(w.steps)]
        mk.sync()
        runs.append((torch.stack(outs), mk.view(0)["pos"].clone(), mk.view(0)["ring_c"].clone()))
        mk.close()
    for r in runs[1:]:
        assert torch.equal(r[0], runs[0][0]) and torch.equal(r[1], runs[0][1]) and torch.equal(r[2], runs[0][2])


# ---- batch rows with prompts of different lengths
@pytest.mark.parametrize("kernel,dtype,d", [("tc", "bf16", 128), ("simt", "bf16", 128), ("simt", "f32", 64)])
def test_ragged_prompt_lengths_per_batch_row(kernel, dtype, d):
    # C + R = 216: row 0 starts full and evicts from the first step, row 1 reaches capacity after 66 steps, row 2
    # starts shorter than the window, row 3 is the longest and sets the common time axis
    w = synth.Workload("ragged", 2, 4, 8, 2, d, dtype, 0, 90, 200, 16, "sum", 606)
    rep = run_parity_ragged(w, [300, 150, 9, 411], steps=w.steps, kernel=kernel)
    _report(rep)
    assert rep.kernel == kernel and rep.units == 16
    assert rep.evictions == 4 * (90 + 24 + 0 + 90)        # 4 units per row


def test_ragged_rows_with_per_layer_calls_layer_aware_and_current_normalisation():
    w = synth.Workload("ragged2", 3, 3, 14, 2, 128, "bf16", 0, 40, 120, 12, "max", 607)      # group 7 -> 8
    rep = run_parity_ragged(w, [140, 77, 200], steps=w.steps, kernel="auto", per_layer=2)
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0
    rep = run_parity_ragged(w, [140, 77, 200], steps=w.steps, kernel="auto", full_layers=1, max_tokens=256)
    _report(rep)
    assert rep.evictions > 0
    rep = run_parity_ragged(w, [140, 77, 200], steps=w.steps, kernel="auto", norm="current")
    _report(rep)
    assert rep.evictions > 0


def test_ragged_prefill_rejects_what_it_does_not_support():
    mk = binding.MorphKV(1, 2, 8, 2, 128, 64, 16, "sum", "bf16", evict_interval=4)
    k = torch.zeros((1, 2, 2, 100, 128), dtype=torch.bfloat16, device="cuda:0")
    q = torch.zeros((1, 2, 8, 16, 128), dtype=torch.bfloat16, device="cuda:0")
    assert binding.mkv_prefill_ragged(mk.ctx, k, k, q, [100, 50], 100) == binding.UNSUPPORTED
    mk.close()
    mk = binding.MorphKV(1, 2, 8, 2, 128, 64, 16, "sum", "bf16")
    assert binding.mkv_prefill_ragged(mk.ctx, k, k, q, [100, 101], 100) == binding.INVALID_ARG
    assert binding.mkv_prefill_ragged(mk.ctx, k, k, q, [100, 0], 100) == binding.INVALID_ARG
    mk.close()


# ---- the step index lives on the device: steps recorded in a CUDA graph and replayed
@pytest.mark.parametrize("kernel,dtype,d,profile,T", [("tc", "bf16", 128, "recompute", 1), ("simt", "f32", 64, "recompute", 1),
                                                      ("tc", "bf16", 128, "stored", 1), ("tc", "bf16", 128, "recompute", 3)])
def test_steps_replayed_from_a_cuda_graph_equal_direct_calls(kernel, dtype, d, profile, T):
    # Four steps are captured once (launches only, on a side stream) and replayed three times with fresh inputs in
    # the same buffers; a second context takes the same twelve steps by direct calls.  Outputs bit for bit, the
    # same retained positions, and the host mirror follows the device state after mkv_sync.  The cache fills
    # during the first replays and evicts afterwards, so the graph's launches meet both kinds of step.
    w = synth.Workload("graph", 2, 2, 8, 2, d, dtype, 90, 12, 80, 16, "max", 808)
    dev = torch.device("cuda:0")
    tdt = synth.torch_dtype(dtype)
    st = synth.Stream(w, dev)
    P, S, reps = w.prompt_len, 4, 3
    k, v = st.kv(np.arange(P))
    qw = st.q(np.arange(P - w.R, P))
    kk, vv = st.kv(np.arange(P, P + S * reps))
    qq = st.q(np.arange(P, P + S * reps))
    qs = qq.permute(3, 0, 1, 2, 4).to(tdt).contiguous()        # [steps, L, B, Hq, d]
    ks = kk.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
    vs = vv.permute(3, 0, 1, 2, 4).to(tdt).contiguous()

    def fresh():
        # (T = 3 against four recorded steps: every replay meets the eviction period in another phase)
        mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, d, w.C, w.R, w.fusion, dtype, kernel=kernel,
                             profile=profile, evict_interval=T)
        mk.prefill(k.to(tdt).contiguous(), v.to(tdt).contiguous(), qw.to(tdt).contiguous())
        mk.sync()
        return mk

    direct = fresh()
    want = torch.empty_like(qs)
    for i in range(S * reps):
        direct.decode_step(qs[i], ks[i], vs[i], want[i])
    direct.sync()

    mk = fresh()
    q_in, k_in, v_in = torch.empty_like(qs[:S]), torch.empty_like(ks[:S]), torch.empty_like(vs[:S])
    out = torch.empty_like(qs[:S])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for i in range(S):
            mk.decode_step(q_in[i], k_in[i], v_in[i], out[i], stream=torch.cuda.current_stream())
    # the capture enqueued nothing: the context's host mirror ran ahead by S steps, the device did not
    mk.sync()
    got = torch.empty_like(qs)
    for r in range(reps):
        q_in.copy_(qs[r * S:(r + 1) * S]); k_in.copy_(ks[r * S:(r + 1) * S]); v_in.copy_(vs[r * S:(r + 1) * S])
        g.replay()
        torch.cuda.synchronize()
        got[r * S:(r + 1) * S] = out
    mk.sync()
    assert torch.equal(got, want)
    for l in range(w.layers):
        a, b = mk.view(l), direct.view(l)
        assert a["count"] == b["count"] and a["next_pos"] == b["next_pos"] == P + S * reps
        assert torch.equal(torch.sort(a["pos"][:, :, :a["count"]], dim=-1).values, torch.sort(b["pos"][:, :, :b["count"]], dim=-1).values)
    mk.close()
    direct.close()


def test_reset_after_ragged_prompts_gives_a_uniform_context_again():
    # a context that held rows of different lengths, reset and loaded with one uniform prompt, behaves like a fresh one
    w = synth.Workload("ragged_reset", 2, 3, 8, 2, 128, "bf16", 150, 6, 100, 16, "sum", 611)
    dev = torch.device("cuda:0")
    st = synth.Stream(w, dev)
    P = w.prompt_len
    k, v = st.kv(np.arange(P))
    qw = st.q(np.arange(P - w.R, P))
    kb, vb, qb = k.bfloat16().contiguous(), v.bfloat16().contiguous(), qw.bfloat16().contiguous()
    kk, vv = st.kv(np.arange(P, P + w.steps))
    qq = st.q(np.arange(P, P + w.steps))

    def steps(mk):
        outs = []
        for i in range(w.steps):
            outs.append(mk.decode_step(qq[..., i, :].bfloat16().contiguous(), kk[..., i, :].bfloat16().contiguous(),
                                       vv[..., i, :].bfloat16().contiguous()).clone())
        mk.sync()
        return torch.stack(outs), [torch.sort(mk.view(l)["pos"][:, :, :mk.view(l)["count"]], dim=-1).values.clone() for l in range(w.layers)]

    fresh = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, 128, w.C, w.R, w.fusion, "bf16")
    fresh.prefill(kb, vb, qb)
    want = steps(fresh)
    fresh.close()
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, 128, w.C, w.R, w.fusion, "bf16")
    mk.prefill_ragged(kb, vb, qb, [150, 60, 97])
    mk.decode_step(qq[..., 0, :].bfloat16().contiguous(), kk[..., 0, :].bfloat16().contiguous(), vv[..., 0, :].bfloat16().contiguous())
    mk.sync()
    cnt, nxt = mk.row_state(0)
    assert nxt == [151, 61, 98] and cnt == [116, 61, 98]
    mk.reset()
    mk.prefill(kb, vb, qb)
    got = steps(mk)
    cnt, nxt = mk.row_state(1)
    assert nxt == [P + w.steps] * 3 and cnt == [w.C + w.R] * 3
    mk.close()
    assert torch.equal(got[0], want[0])
    assert all(torch.equal(a, b) for a, b in zip(got[1], want[1]))


@pytest.mark.parametrize("lens", [[5, 9, 3], [7], [40, 40, 40]])
def test_ragged_prompts_degenerate_cases(lens):
    # every prompt shorter than the window (the padded tensors are then shorter than R too), a batch of one row, and
    # rows that happen to be equally long
    w = synth.Workload("ragged_edge", 2, len(lens), 8, 2, 128, "bf16", 0, 50, 30, 16, "sum", 612)
    rep = run_parity_ragged(w, lens, steps=w.steps, kernel="auto")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0


# ---- the attention profiles kept as a table beside the cache (the paper's own bookkeeping) instead of recomputed
@pytest.mark.parametrize("q_heads,kv_heads,R,C,P,fusion", [(8, 2, 16, 150, 260, "sum"),      # evicts from the first step
                                                           (8, 2, 32, 230, 200, "max"),      # starts in the fill phase
                                                           (14, 2, 12, 90, 133, "sum"),      # group 7 -> 8
                                                           (8, 2, 200, 600, 1000, "sum"),    # window 200: 800 ring rows
                                                           (2, 2, 9, 40, 5, "max"),          # prompt shorter than the window
                                                           (8, 2, 700, 900, 1200, "sum")])   # window 700: beyond what recomputation takes
def test_stored_profile_mode(q_heads, kv_heads, R, C, P, fusion):
    w = synth.Workload("stored", 2, 2, q_heads, kv_heads, 128, "bf16", P, 2 * R + 40, C, R, fusion, 900 + R)
    rep = run_parity(w, steps=w.steps, n_units=8, kernel="auto", check_F_every=5, profile="stored")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0


def test_stored_profile_mode_with_per_layer_calls_and_reset():
    w = synth.Workload("stored_layer", 3, 1, 8, 2, 128, "bf16", 300, 40, 200, 24, "sum", 951)
    rep = run_parity(w, steps=w.steps, n_units=6, kernel="auto", per_layer=2, profile="stored")
    _report(rep)
    assert rep.kernel == "tc" and rep.evictions > 0
    p = binding.mkv_default_params()
    p.layers, p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.C, p.R = 1, 1, 8, 2, 64, 64, 16       # head_dim 64: CUDA-core kernel only
    p.profile_mode = binding.PROFILE["stored"]
    st, h = binding.mkv_create_ex(p)
    assert st == binding.UNSUPPORTED and h is None
