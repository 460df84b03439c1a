"""Lock-step parity harness: the CUDA path (through the C ABI) against the CPU oracle.

Both sides receive the same materialised tensors.  Per decode step and per checked unit the
harness compares the attention output (max abs error) and the evicted position.  Where the
device evicts a different token than the oracle ranks last, the choice is accepted only if
the oracle's own fused scores of the two tokens are a near tie (relative gap <= 1e-3, or
both below 1e-30); the oracle is then made to follow the device so later steps stay
comparable.  Anything else is a failure.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle import morphkv_oracle as ora
from paper_2503_00979_b200 import binding, synth

TOL_OUT = {"bf16": 2e-2, "f32": 1e-4}     # max abs error of attention outputs, per step
TIE_REL = 1e-3
TIE_FLOOR = 1e-30


@dataclasses.dataclass
class ParityReport:
    steps: int = 0
    unit_steps: int = 0
    max_out_err: float = 0.0
    evictions: int = 0
    near_tie_resyncs: int = 0
    max_F_rel_err: float = 0.0
    F_compared: int = 0
    prefill_dropped: int = 0
    kernel: str = ""


def near_tie(a: float, b: float) -> bool:
    if abs(a) < TIE_FLOOR and abs(b) < TIE_FLOOR:
        return True
    return abs(a - b) <= TIE_REL * max(abs(a), abs(b))


def pick_units(w: synth.Workload, n: int, seed: int = 0):
    """First and last unit plus a seeded sample, as (layer, batch row, kv head) triples."""
    all_units = [(l, b, h) for l in range(w.layers) for b in range(w.batch) for h in range(w.n_kv_heads)]
    if n >= len(all_units):
        return all_units
    rng = np.random.default_rng(seed)
    idx = {0, len(all_units) - 1} | set(rng.choice(len(all_units), size=n, replace=False).tolist())
    return [all_units[i] for i in sorted(idx)][:max(n, 2)]


def run_parity(w: synth.Workload, steps: int, units=None, n_units: int = 8, chunk: int = 32, kernel: str = "auto",
               splits: int = 0, check_F_every: int = 16, device: str = "cuda:0", use_steps_call: bool = False,
               host_call_every: int = 0, host_pinned: bool = True) -> ParityReport:
    dev = torch.device(device)
    st = synth.Stream(w, dev)
    tdt = synth.torch_dtype(w.dtype)
    G, d, P, R, C_ = w.group, w.head_dim, w.prompt_len, w.R, w.C
    units = units or pick_units(w, n_units)
    rep = ParityReport()
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, d, C_, R, w.fusion, w.dtype, kernel=kernel,
                         splits=splits, device=device)
    rep.kernel = mk.kernel_name
    tol = TOL_OUT[w.dtype]
    Rw = min(R, P)

    # ---- prefill: inputs are drawn layer by layer so that full-size workloads fit in memory ----
    Hkv, Hq = w.n_kv_heads, w.n_q_heads
    k_all = torch.empty((w.layers, w.batch, Hkv, P, d), dtype=tdt, device=dev)
    v_all = torch.empty_like(k_all)
    qw_all = torch.empty((w.layers, w.batch, Hq, Rw, d), dtype=tdt, device=dev)
    prompt = {}
    for l in range(w.layers):
        k32, v32 = st.kv(np.arange(P), [l])
        qw32 = st.q(np.arange(P - Rw, P), [l])
        k_all[l], v_all[l], qw_all[l] = k32[0].to(tdt), v32[0].to(tdt), qw32[0].to(tdt)
        for (ul, b, h) in units:
            if ul == l:
                prompt[(ul, b, h)] = (k32[0, b, h].double().cpu().numpy(), v32[0, b, h].double().cpu().numpy(),
                                      qw32[0, b, h * G:(h + 1) * G].double().cpu().numpy(), k32[0, b, h].clone())
        del k32, v32, qw32
    mk.prefill(k_all, v_all, qw_all)
    mk.sync()
    del k_all, v_all, qw_all
    orac = {}
    for (l, b, h) in units:
        kp, vp, qp, k_dev = prompt[(l, b, h)]
        u = ora.Unit(G, d, C_, R, w.fusion)
        u.prefill(kp, vp, qp)
        view = mk.view(l)
        gp = view["pos"][b, h, :view["count"]].cpu().numpy()
        assert view["count"] == u.count, (view["count"], u.count)
        if set(gp.tolist()) != set(u.positions().tolist()):
            kth, k1 = u.last_boundary()
            assert near_tie(kth, k1), f"prefill retained set differs for unit {(l, b, h)} without a near tie"
            rep.prefill_dropped += 1
            continue
        # K/V rows must be the prompt rows of those positions, bit for bit
        kk = view["K"][b, h, :view["count"]].float().cpu()
        assert torch.equal(kk, k_dev[torch.from_numpy(gp).long().to(dev)].cpu())
        orac[(l, b, h)] = u
    del prompt

    # ---- decode in chunks ----
    done = 0
    while done < steps:
        ns = min(chunk, steps - done)
        pos = np.arange(P + done, P + done + ns)
        k32, v32 = st.kv(pos)                 # [L,B,Hkv,ns,d]
        q32 = st.q(pos)                       # [L,B,Hq,ns,d]
        qs = q32.permute(3, 0, 1, 2, 4).to(tdt).contiguous()    # [ns,L,B,Hq,d]
        ks = k32.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
        vs = v32.permute(3, 0, 1, 2, 4).to(tdt).contiguous()
        outs = torch.empty_like(qs)
        evh = torch.empty((ns, w.layers, w.batch, w.n_kv_heads), dtype=torch.int32, device=dev)
        Fsnap = {}
        if use_steps_call:
            mk.decode_steps(qs, ks, vs, outs)
            evh = None
        else:
            for i in range(ns):
                if host_call_every and (done + i) % host_call_every == 0:
                    qh, kh, vh = qs[i].cpu(), ks[i].cpu(), vs[i].cpu()
                    oh = torch.empty_like(qh)
                    if host_pinned:
                        qh, kh, vh, oh = qh.pin_memory(), kh.pin_memory(), vh.pin_memory(), oh.pin_memory()
                    mk.decode_step_host(qh, kh, vh, oh)
                    torch.cuda.current_stream().synchronize()
                    outs[i].copy_(oh)
                else:
                    mk.decode_step(qs[i], ks[i], vs[i], outs[i])
                for l in sorted({u[0] for u in orac}):
                    evh[i, l].copy_(mk.view(l)["evicted_pos"])
                if check_F_every and (done + i) % check_F_every == check_F_every - 1:
                    Fsnap[i] = {l: (mk.view(l)["F"].clone(), mk.view(l)["pos"].clone()) for l in {u[0] for u in orac}}
        mk.sync()
        outs_c = outs.float().cpu().numpy()
        q_c, k_c, v_c = q32.double().cpu().numpy(), k32.double().cpu().numpy(), v32.double().cpu().numpy()
        ev_c = evh.cpu().numpy() if evh is not None else None
        for (l, b, h), u in orac.items():
            for i in range(ns):
                t = P + done + i
                e_g = int(ev_c[i, l, b, h]) if ev_c is not None else None
                forced = [e_g] if (e_g is not None and e_g >= 0) else None
                o = u.step(q_c[l, b, h * G:(h + 1) * G, i], k_c[l, b, h, i], v_c[l, b, h, i], forced=forced)
                err = float(np.abs(o - outs_c[i, l, b, h * G:(h + 1) * G]).max())
                rep.max_out_err = max(rep.max_out_err, err)
                assert err <= tol, f"unit {(l, b, h)} step {t}: attention output error {err:.3e} > {tol}"
                cp, cF = u.last_scores()
                if ev_c is not None:
                    if len(cp) > C_:
                        rep.evictions += 1
                        assert e_g >= 0, f"unit {(l, b, h)} step {t}: device did not evict"
                        own = int(cp[C_])
                        if e_g != own:
                            Fg = float(cF[np.nonzero(cp == e_g)[0][0]])
                            assert near_tie(Fg, float(cF[C_])), \
                                (f"unit {(l, b, h)} step {t}: device evicted {e_g} (F={Fg:.6e}) but the oracle ranks "
                                 f"{own} last (F={cF[C_]:.6e}), no near tie")
                            rep.near_tie_resyncs += 1
                    else:
                        assert e_g == -1, f"unit {(l, b, h)} step {t}: device evicted {e_g} but the cache is not full"
                if i in Fsnap and len(cp) > C_:
                    Fg_all, pos_all = Fsnap[i][l]
                    Fg_u = Fg_all[b, h].cpu().numpy()
                    # the snapshot is taken after the step: the evicted slot now holds position t
                    pos_u = pos_all[b, h].cpu().numpy()
                    lut = {int(p): float(f) for p, f in zip(pos_u, Fg_u)}
                    for p, f in zip(cp, cF):
                        if int(p) in lut and lut[int(p)] >= 0 and f > 1e-20:
                            rep.max_F_rel_err = max(rep.max_F_rel_err, abs(lut[int(p)] - f) / f)
                            rep.F_compared += 1
                rep.unit_steps += 1
            gpos = mk.view(l)["pos"][b, h, :mk.view(l)["count"]].cpu().numpy()
            if ev_c is not None:
                assert set(gpos.tolist()) == set(u.positions().tolist()), f"unit {(l, b, h)}: retained sets differ"
        done += ns
        rep.steps = done
    if rep.F_compared:
        assert rep.max_F_rel_err < 1e-3, f"fused scores off by {rep.max_F_rel_err:.3e} relative"
    mk.close()
    return rep


def run_parity_coarse(w: synth.Workload, T: int, steps: int, n_units: int = 4, kernel: str = "auto",
                      device: str = "cuda:0") -> ParityReport:
    """Lock-step parity for coarse-grained eviction (the policy runs every T-th step and may drop several
    tokens at once).  After every step the retained position set of each checked unit is read back; what the
    device dropped is the oracle's set before the step, plus the new token, minus that.  The oracle is made
    to drop the same tokens, and wherever that differs from its own ranking every token in the difference
    must be a near tie with the boundary of its top C."""
    dev = torch.device(device)
    st = synth.Stream(w, dev)
    tdt = synth.torch_dtype(w.dtype)
    G, d, P, R, C_ = w.group, w.head_dim, w.prompt_len, w.R, w.C
    units = pick_units(w, n_units)
    rep = ParityReport()
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, d, C_, R, w.fusion, w.dtype, evict_interval=T,
                         kernel=kernel, device=device)
    rep.kernel = mk.kernel_name
    tol = TOL_OUT[w.dtype]
    Rw = min(R, P)
    k32, v32 = st.kv(np.arange(P))
    qw32 = st.q(np.arange(P - Rw, P))
    mk.prefill(k32.to(tdt).contiguous(), v32.to(tdt).contiguous(), qw32.to(tdt).contiguous())
    mk.sync()
    orac = {}
    for (l, b, h) in units:
        u = ora.Unit(G, d, C_, R, w.fusion, evict_interval=T)
        u.prefill(k32[l, b, h].double().cpu().numpy(), v32[l, b, h].double().cpu().numpy(),
                  qw32[l, b, h * G:(h + 1) * G].double().cpu().numpy())
        view = mk.view(l)
        gp = set(view["pos"][b, h, :view["count"]].cpu().numpy().tolist())
        if gp != set(u.positions().tolist()):
            kth, k1 = u.last_boundary()
            assert near_tie(kth, k1), f"prefill retained set differs for unit {(l, b, h)} without a near tie"
            rep.prefill_dropped += 1
            continue
        orac[(l, b, h)] = u
    peak = 0
    for i in range(steps):
        t = P + i
        k1_, v1_ = st.kv([t])
        q1_ = st.q([t])
        qs = q1_[..., 0, :].to(tdt).contiguous()
        ks = k1_[..., 0, :].to(tdt).contiguous()
        vs = v1_[..., 0, :].to(tdt).contiguous()
        out = torch.empty_like(qs)
        mk.decode_step(qs, ks, vs, out)
        mk.sync()
        out_c = out.float().cpu().numpy()
        q_c, k_c, v_c = q1_.double().cpu().numpy(), k1_.double().cpu().numpy(), v1_.double().cpu().numpy()
        views = {l: mk.view(l) for l in {u_[0] for u_ in orac}}
        for (l, b, h), u in orac.items():
            view = views[l]
            peak = max(peak, view["count"])
            gp = set(view["pos"][b, h, :view["count"]].cpu().numpy().tolist())
            assert len(gp) == view["count"] and -1 not in gp, f"unit {(l, b, h)} step {t}: slots are not a dense prefix"
            before = set(u.positions().tolist()) | {t}
            dropped = sorted(before - gp)
            assert gp <= before, f"unit {(l, b, h)} step {t}: device holds tokens the oracle never had"
            o = u.step(q_c[l, b, h * G:(h + 1) * G, 0], k_c[l, b, h, 0], v_c[l, b, h, 0], forced=dropped or None)
            err = float(np.abs(o - out_c[l, b, h * G:(h + 1) * G]).max())
            rep.max_out_err = max(rep.max_out_err, err)
            assert err <= tol, f"unit {(l, b, h)} step {t}: attention output error {err:.3e} > {tol}"
            cp, cF = u.last_scores()
            if len(cp) > C_:
                rep.evictions += len(dropped)
                assert len(dropped) == len(cp) - C_, (f"unit {(l, b, h)} step {t}: device dropped {len(dropped)} tokens, "
                                                      f"the policy drops {len(cp) - C_}")
                own = set(int(p) for p in cp[C_:])
                diff = own ^ set(dropped)
                if diff:
                    Fof = {int(p): float(f) for p, f in zip(cp, cF)}
                    for x in diff:
                        assert near_tie(Fof[x], float(cF[C_ - 1])) or near_tie(Fof[x], float(cF[C_])), \
                            f"unit {(l, b, h)} step {t}: token {x} (F={Fof[x]:.6e}) changed sides without a near tie"
                    rep.near_tie_resyncs += 1
            else:
                assert not dropped, f"unit {(l, b, h)} step {t}: device dropped {dropped} on a step without the policy"
            assert set(u.positions().tolist()) == gp, f"unit {(l, b, h)} step {t}: retained sets differ"
            # K rows of the retained tokens are the rows that were appended, bit for bit
            rep.unit_steps += 1
        rep.steps = i + 1
    rep.F_compared = peak        # reused: the largest fill seen (C + R + T - 1 expected)
    mk.close()
    return rep
