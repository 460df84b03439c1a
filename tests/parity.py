"""Lock-step parity harness: the CUDA path (through the C ABI) against the CPU oracle.

Both sides receive the same materialised tensors.  Per decode step and per checked unit the
harness compares the attention output (max abs error) and the evicted position.  Where the
device evicts a different token than the oracle ranks last, the choice is accepted only if
the oracle's own fused scores of the two tokens are a near tie (relative gap <= 1e-3); the
oracle is then made to follow the device so later steps stay comparable.  Anything else is a
failure.  The same rule covers the prompt phase: a retained set that differs from the
oracle's must differ only in tokens whose fused scores tie with the boundary of the top C,
and the oracle then starts from the device's set.

The oracle units are independent, so their steps run on a thread pool (the C calls release
the interpreter lock); only the sampled units' inputs are converted to float64.
"""
from __future__ import annotations

import dataclasses
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

from oracle import morphkv_oracle as ora
from paper_2503_00979_b200 import binding, synth

TOL_OUT = {"bf16": 2e-2, "f32": 1e-4}     # max abs error of attention outputs, per step
TIE_REL = 1e-3


@dataclasses.dataclass
class ParityReport:
    steps: int = 0
    unit_steps: int = 0
    units: int = 0
    max_out_err: float = 0.0
    evictions: int = 0
    near_tie_resyncs: int = 0           # decode steps on which the device's choice differed within the tie rule
    prefill_resyncs: int = 0            # units whose prompt-phase set differed within the tie rule
    min_rel_gap: float = float("inf")   # smallest relative gap between the oracle's C-th and (C+1)-th score
    max_F_rel_err: float = 0.0
    F_compared: int = 0
    kernel: str = ""


def near_tie(a: float, b: float) -> bool:
    return abs(a - b) <= TIE_REL * max(abs(a), abs(b))


def rel_gap(a: float, b: float) -> float:
    m = max(abs(a), abs(b))
    return abs(a - b) / m if m > 0 else 0.0


def pick_units(w: synth.Workload, n: int, seed: int = 0):
    """First and last unit plus a seeded sample, as (layer, batch row, kv head) triples."""
    all_units = [(l, b, h) for l in range(w.layers) for b in range(w.batch) for h in range(w.n_kv_heads)]
    if n >= len(all_units):
        return all_units
    rng = np.random.default_rng(seed)
    idx = {0, len(all_units) - 1} | set(rng.choice(len(all_units), size=n, replace=False).tolist())
    return [all_units[i] for i in sorted(idx)][:max(n, 2)]


def _workers() -> int:
    return max(1, min(32, len(os.sched_getaffinity(0))))


def _f64(t: torch.Tensor) -> np.ndarray:
    return t.double().cpu().numpy()


class _DeviceStream:
    """synth.Stream whose draws are made on one device and delivered on another."""

    def __init__(self, w, draw_on, deliver_on):
        self.st, self.to = synth.Stream(w, draw_on), torch.device(deliver_on)

    def kv(self, *a, **k):
        x, y = self.st.kv(*a, **k)
        return x.to(self.to), y.to(self.to)

    def q(self, *a, **k):
        return self.st.q(*a, **k).to(self.to)


def oracle_unit_following(make_unit, k, v, qw, device_positions, where: str):
    """A prefilled oracle unit (from `make_unit()`) whose retained set equals the device's.  If the oracle's own
    choice differs, every token that changed sides must tie with the boundary of its top C, and the oracle is
    prefilled again with the device's evictions forced.  Returns (unit, resynced)."""
    u = make_unit()
    u.prefill(k, v, qw)
    dev = set(int(p) for p in device_positions)
    own = set(u.positions().tolist())
    if dev == own:
        return u, False
    cp, cF = u.last_scores()
    assert len(cp) > u.C, f"{where}: prompt-phase sets differ although nothing had to be evicted"
    Fof = {int(p): float(f) for p, f in zip(cp, cF)}
    kth, k1 = float(cF[u.C - 1]), float(cF[u.C])
    for p in dev ^ own:
        assert p in Fof, f"{where}: prompt position {p} is not a candidate"
        assert near_tie(Fof[p], kth) or near_tie(Fof[p], k1), \
            f"{where}: prompt token {p} (F={Fof[p]:.6e}) changed sides without a near tie (boundary {kth:.6e} / {k1:.6e})"
    u2 = make_unit()
    u2.prefill(k, v, qw, forced=sorted(set(int(p) for p in cp) - dev))
    assert set(u2.positions().tolist()) == dev
    return u2, True


def run_parity(w: synth.Workload, steps: int, units=None, n_units: int = 8, chunk: int = 32, kernel: str = "auto",
               splits: int = 0, check_F_every: int = 16, device: str = "cuda:0", use_steps_call: bool = False,
               host_call_every: int = 0, host_pinned: bool = True, synth_device=None, per_layer: int = 0,
               full_layers: int = 0, max_tokens: int = 0, norm: str = "frozen", **ctx_kwargs) -> ParityReport:
    """Prefill + `steps` decode steps of workload `w` on the device, followed by the oracle on `units`.

    The steps of a chunk are enqueued without a synchronisation in between (the evicted positions of the
    checked units are gathered on the stream and read back once per chunk).
    use_steps_call   one mkv_decode_steps call per chunk (no per-step evicted positions: outputs are compared on
                     every step, retained sets at the end of each chunk unless the oracle saw a near tie in it).
    synth_device     where the inputs are drawn ("cpu" keeps the drawing's many small kernels off the GPU).
    per_layer        1: every step is made of mkv_decode_step_layer calls, layer by layer; 2: steps alternate between
                     one whole-stack call and per-layer calls.
    norm             "frozen" (default) or "current": how window rows' weights are normalised, on both sides.
    full_layers, max_tokens   layer-aware variant: the first full_layers layers keep every token (the oracle units of
                     those layers get C = max_tokens - R, so they never evict within max_tokens).
    """
    dev = torch.device(device)
    st = _DeviceStream(w, synth_device or dev, dev)
    tdt = synth.torch_dtype(w.dtype)
    G, d, P, R, C_ = w.group, w.head_dim, w.prompt_len, w.R, w.C
    units = units or pick_units(w, n_units)
    rep = ParityReport()
    mk = binding.MorphKV(w.layers, w.batch, w.n_q_heads, w.n_kv_heads, d, C_, R, w.fusion, w.dtype, kernel=kernel,
                         splits=splits, device=device, full_layers=full_layers, max_tokens=max_tokens, norm=norm,
                         **ctx_kwargs)
    rep.kernel = mk.kernel_name
    C_of = {l: (max_tokens - R if l < full_layers else C_) for l in range(w.layers)}     # distant tokens kept per layer
    tol = TOL_OUT[w.dtype]
    Rw = min(R, P)
    pool = ThreadPoolExecutor(max_workers=_workers())

    # ---- prefill: inputs are drawn layer by layer so that full-size workloads fit in memory ----
    Hkv, Hq = w.n_kv_heads, w.n_q_heads
    k_all = torch.empty((w.layers, w.batch, Hkv, P, d), dtype=tdt, device=dev)
    v_all = torch.empty_like(k_all)
    qw_all = torch.empty((w.layers, w.batch, Hq, Rw, d), dtype=tdt, device=dev)
    by_layer = {}
    for (l, b, h) in units:
        by_layer.setdefault(l, []).append((b, h))
    prompt = {}
    for l in range(w.layers):
        k32, v32 = st.kv(np.arange(P), [l])
        qw32 = st.q(np.arange(P - Rw, P), [l])
        k_all[l], v_all[l], qw_all[l] = k32[0].to(tdt), v32[0].to(tdt), qw32[0].to(tdt)
        for (b, h) in by_layer.get(l, []):
            prompt[(l, b, h)] = (_f64(k32[0, b, h]), _f64(v32[0, b, h]), _f64(qw32[0, b, h * G:(h + 1) * G]))
        del k32, v32, qw32
    mk.prefill(k_all, v_all, qw_all)
    mk.sync()
    views = {l: mk.view(l) for l in by_layer}
    count0 = {l: views[l]["count"] for l in by_layer}
    dev_pos = {(l, b, h): views[l]["pos"][b, h, :count0[l]].cpu().numpy() for (l, b, h) in units}

    def prefill_unit(key):
        kp, vp, qp = prompt[key]
        u, resync = oracle_unit_following(lambda: ora.Unit(G, d, C_of[key[0]], R, w.fusion, norm=norm), kp, vp, qp, dev_pos[key], f"unit {key}")
        assert count0[key[0]] == u.count, (count0[key[0]], u.count)
        return key, u, resync

    orac = {}
    for key, u, resync in pool.map(prefill_unit, units):
        orac[key] = u
        rep.prefill_resyncs += int(resync)
    # K rows must be the prompt rows of those positions, bit for bit
    for (l, b, h) in units:
        gp = torch.from_numpy(dev_pos[(l, b, h)]).long().to(dev)
        assert torch.equal(views[l]["K"][b, h, :count0[l]], k_all[l, b, h][gp]), f"unit {(l, b, h)}: K rows differ from the prompt's"
        assert torch.equal(views[l]["V"][b, h, :count0[l]], v_all[l, b, h][gp]), f"unit {(l, b, h)}: V rows differ from the prompt's"
    del k_all, v_all, qw_all, prompt
    rep.units = len(orac)
    layers_checked = sorted(by_layer)
    li = torch.tensor([l for (l, b, h) in units], device=dev)
    bi = torch.tensor([b for (l, b, h) in units], device=dev)
    hi = torch.tensor([h for (l, b, h) in units], device=dev)
    lidx = torch.tensor([layers_checked.index(l) for (l, b, h) in units], device=dev)

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
        evh = torch.empty((ns, len(units)), dtype=torch.int32, device=dev)
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
                elif per_layer == 1 or (per_layer == 2 and (done + i) % 2 == 1):
                    for l in range(w.layers):
                        mk.decode_step_layer(l, qs[i, l], ks[i, l], vs[i, l], outs[i, l])
                else:
                    mk.decode_step(qs[i], ks[i], vs[i], outs[i])
                # evicted positions of the checked units, gathered on the stream
                ev_all = torch.stack([views[l]["evicted_pos"] for l in layers_checked])      # [layers checked, B, Hkv]
                evh[i] = ev_all[lidx, bi, hi]
                if check_F_every and (done + i) % check_F_every == check_F_every - 1:
                    Fsnap[i] = {l: (views[l]["F"].clone(), views[l]["pos"].clone()) for l in layers_checked}
        mk.sync()
        # only the checked units cross to the host
        q_u = _f64(q32.view(w.layers, w.batch, Hkv, G, ns, d)[li, bi, hi])        # [units, G, ns, d]
        k_u, v_u = _f64(k32[li, bi, hi]), _f64(v32[li, bi, hi])                     # [units, ns, d]
        o_u = outs.view(ns, w.layers, w.batch, Hkv, G, d)[:, li, bi, hi].float().cpu().numpy()   # [ns, units, G, d]
        ev_c = evh.cpu().numpy() if evh is not None else None
        del q32, k32, v32, qs, ks, vs, outs
        t0 = P + done

        def follow(ui):
            key = units[ui]
            u = orac[key]
            C_ = C_of[key[0]]
            r = dict(err=0.0, evictions=0, resyncs=0, Fmax=0.0, Fcmp=0, gap=float("inf"))
            for i in range(ns):
                t = t0 + i
                e_g = int(ev_c[i, ui]) if ev_c is not None else None
                forced = [e_g] if (e_g is not None and e_g >= 0) else None
                o = u.step(np.ascontiguousarray(q_u[ui, :, i]), k_u[ui, i], v_u[ui, i], forced=forced)
                err = float(np.abs(o - o_u[i, ui]).max())
                r["err"] = max(r["err"], err)
                assert err <= tol, f"unit {key} step {t}: attention output error {err:.3e} > {tol}"
                cp, cF = u.last_scores()
                if len(cp) > C_:
                    r["gap"] = min(r["gap"], rel_gap(float(cF[C_ - 1]), float(cF[C_])))
                if ev_c is not None:
                    if len(cp) > C_:
                        r["evictions"] += 1
                        assert e_g >= 0, f"unit {key} step {t}: device did not evict"
                        own = int(cp[C_])
                        if e_g != own:
                            Fg = float(cF[np.nonzero(cp == e_g)[0][0]])
                            assert near_tie(Fg, float(cF[C_])), \
                                (f"unit {key} step {t}: device evicted {e_g} (F={Fg:.6e}) but the oracle ranks "
                                 f"{own} last (F={cF[C_]:.6e}), no near tie")
                            r["resyncs"] += 1
                    else:
                        assert e_g == -1, f"unit {key} step {t}: device evicted {e_g} but the cache is not full"
                if i in Fsnap and len(cp) > C_:
                    l, b, h = key
                    Fg_all, pos_all = Fsnap[i][l]
                    Fg_u = Fg_all[b, h].cpu().numpy()
                    # the snapshot is taken after the step: the evicted slot now holds position t
                    pos_u = pos_all[b, h].cpu().numpy()
                    lut = {int(p): float(f) for p, f in zip(pos_u, Fg_u)}
                    for p, f in zip(cp, cF):
                        if int(p) in lut and lut[int(p)] >= 0 and f > 1e-20:
                            r["Fmax"] = max(r["Fmax"], abs(lut[int(p)] - f) / f)
                            r["Fcmp"] += 1
            return r

        results = list(pool.map(follow, range(len(units))))
        gpos = {l: views[l]["pos"][:, :, :mk.view(l)["count"]].cpu().numpy() for l in layers_checked}
        for ui, r in enumerate(results):
            l, b, h = units[ui]
            rep.max_out_err = max(rep.max_out_err, r["err"])
            rep.evictions += r["evictions"]
            rep.near_tie_resyncs += r["resyncs"]
            rep.max_F_rel_err = max(rep.max_F_rel_err, r["Fmax"])
            rep.F_compared += r["Fcmp"]
            rep.min_rel_gap = min(rep.min_rel_gap, r["gap"])
            rep.unit_steps += ns
            same = set(gpos[l][b, h].tolist()) == set(orac[(l, b, h)].positions().tolist())
            if ev_c is not None:
                assert same, f"unit {(l, b, h)}: retained sets differ"
            elif r["gap"] > TIE_REL:
                # no per-step resync in this mode: without a near tie in the chunk the sets must still agree
                assert same, f"unit {(l, b, h)}: retained sets differ after a chunk without a near tie"
        done += ns
        rep.steps = done
    if rep.F_compared:
        assert rep.max_F_rel_err < 1e-3, f"fused scores off by {rep.max_F_rel_err:.3e} relative"
    pool.shutdown()
    mk.close()
    return rep


def run_parity_coarse(w: synth.Workload, T: int, steps: int, n_units: int = 4, kernel: str = "auto",
                      device: str = "cuda:0", synth_device=None) -> ParityReport:
    """Lock-step parity for coarse-grained eviction (the policy runs every T-th step and may drop several
    tokens at once).  After every step the retained position set of each checked unit is read back; what the
    device dropped is the oracle's set before the step, plus the new token, minus that.  The oracle is made
    to drop the same tokens, and wherever that differs from its own ranking every token in the difference
    must be a near tie with the boundary of its top C."""
    dev = torch.device(device)
    st = _DeviceStream(w, synth_device or dev, dev)
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
        view = mk.view(l)
        gp = view["pos"][b, h, :view["count"]].cpu().numpy()
        u, resync = oracle_unit_following(lambda: ora.Unit(G, d, C_, R, w.fusion, evict_interval=T), _f64(k32[l, b, h]),
                                          _f64(v32[l, b, h]), _f64(qw32[l, b, h * G:(h + 1) * G]), gp, f"unit {(l, b, h)}")
        rep.prefill_resyncs += int(resync)
        orac[(l, b, h)] = u
    rep.units = len(orac)
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
            rep.unit_steps += 1
        rep.steps = i + 1
    rep.F_compared = peak        # reused: the largest fill seen (C + R + T - 1 expected)
    mk.close()
    return rep


def run_parity_ragged(w: synth.Workload, prompt_lens, steps: int, kernel: str = "auto", per_layer: int = 0,
                      norm: str = "frozen", device: str = "cuda:0", full_layers: int = 0, max_tokens: int = 0,
                      synth_device=None) -> ParityReport:
    """Lock-step parity for a batch whose rows have prompts of different lengths (`prompt_lens[b]`; `w.prompt_len`
    is ignored).  Every unit of the workload is checked.  Row b's stream is the workload's stream of that row: its
    prompt is positions [0, prompt_lens[b]) and its token of decode step s has position prompt_lens[b] + s, so each
    oracle unit is simply that row's sequence run alone.  The padding of the prompt tensors beyond a row's length
    holds huge values: a kernel that read it would miss the output tolerance at once."""
    dev = torch.device(device)
    st = _DeviceStream(w, synth_device or dev, dev)
    tdt = synth.torch_dtype(w.dtype)
    G, d, R, C_ = w.group, w.head_dim, w.R, w.C
    B, Hkv, L = w.batch, w.n_kv_heads, w.layers
    assert len(prompt_lens) == B
    Pm = max(prompt_lens)
    rep = ParityReport()
    mk = binding.MorphKV(L, B, w.n_q_heads, Hkv, d, C_, R, w.fusion, w.dtype, kernel=kernel, device=device, norm=norm,
                         full_layers=full_layers, max_tokens=max_tokens)
    rep.kernel = mk.kernel_name
    C_of = {l: (max_tokens - R if l < full_layers else C_) for l in range(L)}
    tol = TOL_OUT[w.dtype]
    k32, v32 = st.kv(np.arange(Pm))                       # [L,B,Hkv,Pm,d]
    q32 = st.q(np.arange(Pm))                             # [L,B,Hq,Pm,d]
    qw_len = min(R, Pm)
    k_all, v_all = k32.to(tdt).clone(), v32.to(tdt).clone()
    qw_all = torch.full((L, B, w.n_q_heads, qw_len, d), 1.0e4, dtype=tdt, device=dev)
    for b, P in enumerate(prompt_lens):
        Rw = min(R, P)
        k_all[:, b, :, P:] = 1.0e4
        v_all[:, b, :, P:] = 1.0e4
        qw_all[:, b, :, :Rw] = q32[:, b, :, P - Rw:P].to(tdt)
    mk.prefill_ragged(k_all.contiguous(), v_all.contiguous(), qw_all.contiguous(), list(prompt_lens))
    mk.sync()
    units = [(l, b, h) for l in range(L) for b in range(B) for h in range(Hkv)]
    orac = {}
    for l in range(L):
        view = mk.view(l)
        cnt, nxt = mk.row_state(l)
        assert nxt == list(prompt_lens), (nxt, prompt_lens)
        for b, P in enumerate(prompt_lens):
            Rw = min(R, P)
            assert cnt[b] == (C_of[l] + Rw if P - Rw > C_of[l] else P), (l, b, cnt[b])
            for h in range(Hkv):
                gp = view["pos"][b, h, :cnt[b]].cpu().numpy()
                u, resync = oracle_unit_following(
                    lambda: ora.Unit(G, d, C_of[l], R, w.fusion, norm=norm), _f64(k32[l, b, h, :P]), _f64(v32[l, b, h, :P]),
                    _f64(q32[l, b, h * G:(h + 1) * G, P - Rw:P]), gp, f"unit {(l, b, h)}")
                rep.prefill_resyncs += int(resync)
                idx = torch.from_numpy(gp).long().to(dev)
                assert torch.equal(view["K"][b, h, :cnt[b]], k_all[l, b, h][idx]), f"unit {(l, b, h)}: K rows differ from the prompt's"
                assert torch.equal(view["V"][b, h, :cnt[b]], v_all[l, b, h][idx]), f"unit {(l, b, h)}: V rows differ from the prompt's"
                orac[(l, b, h)] = u
    rep.units = len(orac)
    for i in range(steps):
        # row b's token of this step has position prompt_lens[b] + i
        q1 = torch.empty((L, B, w.n_q_heads, d), dtype=torch.float32, device=dev)
        k1 = torch.empty((L, B, Hkv, d), dtype=torch.float32, device=dev)
        v1 = torch.empty_like(k1)
        for P in sorted(set(prompt_lens)):
            kk, vv = st.kv([P + i])
            qq = st.q([P + i])
            for b in [b for b in range(B) if prompt_lens[b] == P]:
                q1[:, b], k1[:, b], v1[:, b] = qq[:, b, :, 0], kk[:, b, :, 0], vv[:, b, :, 0]
        qs, ks, vs = q1.to(tdt).contiguous(), k1.to(tdt).contiguous(), v1.to(tdt).contiguous()
        out = torch.empty_like(qs)
        if per_layer == 1 or (per_layer == 2 and i % 2 == 1):
            for l in range(L):
                mk.decode_step_layer(l, qs[l], ks[l], vs[l], out[l])
        else:
            mk.decode_step(qs, ks, vs, out)
        mk.sync()
        out_c = out.float().cpu().numpy()
        q_c, k_c, v_c = _f64(q1), _f64(k1), _f64(v1)
        for l in range(L):
            view = mk.view(l)
            cnt, nxt = mk.row_state(l)
            ev = view["evicted_pos"].cpu().numpy()
            pos_l = view["pos"].cpu().numpy()
            for b in range(B):
                t = prompt_lens[b] + i
                assert nxt[b] == t + 1
                for h in range(Hkv):
                    u = orac[(l, b, h)]
                    e_g = int(ev[b, h])
                    o = u.step(np.ascontiguousarray(q_c[l, b, h * G:(h + 1) * G]), k_c[l, b, h], v_c[l, b, h],
                               forced=[e_g] if e_g >= 0 else None)
                    err = float(np.abs(o - out_c[l, b, h * G:(h + 1) * G]).max())
                    rep.max_out_err = max(rep.max_out_err, err)
                    assert err <= tol, f"unit {(l, b, h)} position {t}: attention output error {err:.3e} > {tol}"
                    cp, cF = u.last_scores()
                    if len(cp) > C_of[l]:
                        rep.evictions += 1
                        assert e_g >= 0, f"unit {(l, b, h)} position {t}: device did not evict"
                        own = int(cp[C_of[l]])
                        if e_g != own:
                            Fg = float(cF[np.nonzero(cp == e_g)[0][0]])
                            assert near_tie(Fg, float(cF[C_of[l]])), \
                                f"unit {(l, b, h)} position {t}: device evicted {e_g}, the oracle ranks {own} last, no near tie"
                            rep.near_tie_resyncs += 1
                    else:
                        assert e_g == -1, f"unit {(l, b, h)} position {t}: device evicted {e_g} but the row's cache is not full"
                    assert cnt[b] == u.count, f"unit {(l, b, h)} position {t}: fill {cnt[b]} against the oracle's {u.count}"
                    assert set(pos_l[b, h, :cnt[b]].tolist()) == set(u.positions().tolist()), \
                        f"unit {(l, b, h)} position {t}: retained sets differ"
                    rep.unit_steps += 1
        rep.steps = i + 1
    mk.close()
    return rep
