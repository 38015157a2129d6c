"""Lockstep parity driver: runs the CUDA library and the CPU oracle round by round on the
same seeded synthetic workload and compares them element by element.

Floating-point values (entropy, log-sum-exp, JS divergence and distance, T_G,
P(A|d)) must agree within TOL = 1e-4 absolute.  Discrete results (sampled tokens, stop
flags, window lengths, accept lengths, next tokens, list sizes) must agree exactly,
except where the oracle's own numbers show the decision to be near its threshold:

  * a sampled token whose uniform lies within TIE_EPS of a CDF edge (near-tie),
  * a draft-stop check with |H - T_G| < TOL,
  * an accept draw with |u - P(A|d)| < TOL, or whose outcome changes when d moves by
    +-TOL (the JS distance is the paper's metric; P(A|d) can be steep in d),
  * a vanilla accept draw with |u - alpha| < TOL,
  * a distance within TOL of 0 or 1 (membership of the KDE lists).

Such positions are counted and reported.  After a counted disagreement the GPU state of
that sequence is re-imported from the oracle (never the other way round) so that later
rounds stay comparable.  A disagreement anywhere else raises ParityError.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

import oracle
import synth

TOL = 1e-4
TIE_EPS = 2e-6
# What fp32 can resolve of a JS divergence outside the nearly-equal-rows form: the dominant term
# s log2 s with s close to 2 carries the special-function unit's absolute error of 2^-22, and p, q
# their own rounding.  d = sqrt(D_JS / ln 2) turns an error e of D_JS into e / (2 d ln 2).
JSD_RESOLUTION = 2.5e-7
# The device sums the masses of a top-p decision in double precision, except for bf16 rows, where
# the tokens far below the largest logit are added up from fp32 exponentials: a group of equally
# probable tokens whose decision lies within WARP_BAND of going the other way may be cut on one
# side and kept on the other.  While such groups hold less than WARP_MASS of a row, every
# compared number stays inside its tolerance (H moves by about m |ln m|); a sequence-round with
# more is not compared and the device state is set to the oracle's.
WARP_BAND = {synth.BF16: 5e-7, synth.FP32: 1e-8}
WARP_MASS = 5e-6


def dist_tolerance(d: float) -> float:
    """1e-4, widened only for distances so small that 1e-4 is finer than fp32 resolves D_JS."""
    return max(TOL, JSD_RESOLUTION / (2.0 * max(d, 1e-12) * math.log(2.0))) if d > 0.0 else TOL


class ParityError(AssertionError):
    pass


@dataclass
class Report:
    rounds: int = 0
    positions: int = 0
    draft_rows: int = 0
    near_threshold: int = 0        # flagged decisions met (whether or not they flipped)
    flips: int = 0                 # flagged decisions on which GPU and oracle disagreed
    near_ties: int = 0
    tie_flips: int = 0
    resyncs: int = 0
    r6_resyncs: int = 0            # of those: the flagged position was a distance within TOL of 0 or 1
    dist_checked: int = 0          # distance comparisons made
    dist_beyond_tol: int = 0       # of those: |diff| > TOL, inside what fp32 resolves of D_JS at that distance
    p_acc_checked: int = 0         # P(A|d) comparisons made
    p_acc_beyond_tol: int = 0      # of those: |diff| > TOL, inside the band the steepness of P in d allows
    warp_near: int = 0             # sequence-rounds left out because a top-p cut was too close to call
    max_err: dict = field(default_factory=dict)
    accept_hist: dict = field(default_factory=dict)
    window_hist: dict = field(default_factory=dict)
    vanilla_accept_hist: dict = field(default_factory=dict)
    n_rejections: int = 0

    def err(self, name: str, e: float) -> None:
        if not math.isnan(e):
            self.max_err[name] = max(self.max_err.get(name, 0.0), float(e))

    def summary(self) -> dict:
        counts = dict(rounds=self.rounds, positions=self.positions, draft_rows=self.draft_rows,
                      near_threshold=self.near_threshold, flips=self.flips, near_ties=self.near_ties,
                      tie_flips=self.tie_flips, resyncs=self.resyncs, r6_resyncs=self.r6_resyncs,
                      dist_checked=self.dist_checked, dist_beyond_tol=self.dist_beyond_tol,
                      p_acc_checked=self.p_acc_checked, p_acc_beyond_tol=self.p_acc_beyond_tol, warp_near=self.warp_near,
                      n_rejections=self.n_rejections)
        return dict({k: int(v) for k, v in counts.items()},
                    max_err={k: float(f"{v:.3e}") for k, v in self.max_err.items()},
                    accept_hist=dict(sorted(self.accept_hist.items())),
                    window_hist=dict(sorted(self.window_hist.items())),
                    vanilla_accept_hist=dict(sorted(self.vanilla_accept_hist.items())))


def _bump(h: dict, k: int) -> None:
    h[int(k)] = h.get(int(k), 0) + 1


class Lockstep:
    def __init__(self, wl: synth.Workload, follow: Optional[List[int]] = None,
                 cluster_size: int = 0, list_capacity: Optional[int] = None,
                 min_kde_samples: int = 2, device: int = 0, check_lists_every: int = 16,
                 kde_bandwidth: int = 0, reject_rule: int = 0,
                 warpers: Optional[tuple] = None):
        import torch
        import paper_2512_11280_b200 as adasd
        self.torch, self.adasd, self.wl = torch, adasd, wl
        self.follow = list(range(wl.B)) if follow is None else list(follow)
        self.dev = torch.device("cuda", device)
        cap = list_capacity or max(64, wl.rounds * wl.K + 8)
        self.ctx = adasd.Context(wl.B, wl.V, wl.K, dtype=wl.dtype, list_capacity=cap,
                                 min_kde_samples=min_kde_samples, cluster_size=cluster_size,
                                 kde_bandwidth=kde_bandwidth, reject_rule=reject_rule, device=device)
        # adjusted distribution (temperature, top_k, top_p): set on the context, and applied by
        # the oracle to the host rows before its own steps
        if warpers is not None:                 # as the library stores them: temperature and top_p in fp32
            warpers = (float(np.float32(warpers[0])), int(warpers[1]), float(np.float32(warpers[2])))
            self.ctx.set_warpers(*warpers)
        self.warpers = warpers
        self.gs = synth.GpuSynth(wl, str(self.dev))
        tdt = torch.bfloat16 if wl.dtype == synth.BF16 else torch.float32
        B, K, V = wl.B, wl.K, wl.V
        self.zd = torch.empty((B, K, V), dtype=tdt, device=self.dev)
        self.zt = torch.empty((B, K + 1, V), dtype=tdt, device=self.dev)
        i32 = dict(dtype=torch.int32, device=self.dev)
        f32 = dict(dtype=torch.float32, device=self.dev)
        self.x = torch.zeros((B, K), **i32)
        self.Hk = torch.zeros((K, B), **f32)
        self.lsek = torch.zeros((K, B), **f32)
        self.tokk = torch.zeros((K, B), **i32)
        self.stopk = torch.zeros((K, B), dtype=torch.uint8, device=self.dev)
        self.draft_len = torch.zeros(B, **i32)
        self.active = torch.ones(B, dtype=torch.uint8, device=self.dev)
        self.accept_len = torch.zeros(B, **i32)
        self.next_token = torch.zeros(B, **i32)
        self.v_accept_len = torch.zeros(B, **i32)
        self.v_next_token = torch.zeros(B, **i32)
        self.alpha = torch.zeros((B, K), **f32)
        self.rec = self.ctx.new_record()
        self.states = {b: oracle.SequenceState(capacity=cap + K + 8, min_samples=max(2, min_kde_samples),
                                               bw_rule=kde_bandwidth, reject_rule=reject_rule)
                       for b in self.follow}
        self.reject_rule = reject_rule
        self.report = Report()
        self.check_lists_every = check_lists_every
        # the oracle rounds of the followed sequences run side by side (ctypes releases the GIL);
        # each worker gives the positions of its verify round its share of the host cores
        cores = len(os.sched_getaffinity(0))
        workers = max(1, min(len(self.follow), cores))
        omp = max(1, cores // workers)
        self.pool = ThreadPoolExecutor(max_workers=workers, initializer=lambda: oracle.set_threads(omp))

    # -------------------------------------------------------------- helpers
    def _up(self, a: np.ndarray):
        return self.torch.from_numpy(np.ascontiguousarray(a)).to(self.dev)

    def _fail(self, msg: str):
        raise ParityError(f"[{self.wl.name} round {self.report.rounds}] {msg}")

    def _close(self, name: str, got: float, want: float, tol: float = TOL, ctx: str = ""):
        if math.isnan(want) and math.isnan(got):
            return
        e = abs(got - want)
        self.report.err(name, e)
        if not e <= tol:
            self._fail(f"{name} {ctx}: gpu {got!r} oracle {want!r} |diff| {e:.3e} > {tol:.1e}")

    def _resync(self, b: int) -> None:
        """GPU state of sequence b := the oracle's (after a counted near-threshold flip)."""
        st = self.states[b]
        LE, LA, LR = st.lists()
        self.ctx.state_import(b, st.T_G.value, LE, LA, LR)
        self.report.resyncs += 1

    # -------------------------------------------------------------- one round
    def round(self, r: int) -> None:
        torch, wl, rep = self.torch, self.wl, self.report
        B, K, V = wl.B, wl.K, wl.V
        s_par, t_par = wl.params(r)
        U = synth.round_uniforms_cpu(wl, r)
        u_draft, u_target, u_accept = U["draft"], U["target"], U["accept"]
        g_ud, g_ut, g_ua = self._up(u_draft.T.copy()), self._up(u_target), self._up(u_accept)

        # ---- oracle draft phase for the followed sequences (host rows)
        fb = np.array(self.follow, dtype=np.int32)
        hd, ht = synth.host_round(wl, r, fb)
        skip = set()              # sequences one of whose rows has too much mass on a top-p decision too close to call
        if self.warpers is not None:
            def warp_rows(n):
                d, _, md = oracle.warp(hd[n], *self.warpers, band=WARP_BAND[wl.dtype])
                t, _, mt = oracle.warp(ht[n], *self.warpers, band=WARP_BAND[wl.dtype])
                return d, t, max(md, mt)
            w = list(self.pool.map(warp_rows, range(len(self.follow))))
            hd = np.stack([a[0] for a in w])
            ht = np.stack([a[1] for a in w])
            skip = {self.follow[n] for n, a in enumerate(w) if a[2] > WARP_MASS}
            rep.warp_near += len(skip)
        def draft_phase(n):
            b = self.follow[n]
            st, steps = self.states[b], []
            for k in range(K):
                d = oracle.draft_step(hd[n, k], float(u_draft[b, k]), st.T_G.value)
                steps.append(d)
                if wl.adaptive_window and d["stop"]:
                    break
            return steps
        o_draft = dict(zip(self.follow, self.pool.map(draft_phase, range(len(self.follow)))))

        # ---- GPU draft phase
        self.gs.draft_rows(r, self.zd)
        self.draft_len.zero_()
        self.active.fill_(1)
        for k in range(K):
            self.ctx.draft_entropy(self.zd[:, k, :], self.Hk[k], u=g_ud[k], token_out=self.tokk[k],
                                   active=self.active if wl.adaptive_window else None,
                                   lse_out=self.lsek[k], stop_out=self.stopk[k],
                                   draft_len=self.draft_len, row_stride=K * V)
            if wl.adaptive_window:
                # compare this step now: a flagged stop flip must be repaired before the next step
                stop_h = self.stopk[k].cpu().numpy()
                H_h = self.Hk[k].cpu().numpy()
                for b in self.follow:
                    steps = o_draft[b]
                    if k >= len(steps) or b in skip:
                        continue
                    o = steps[k]
                    self._close("H_draft", float(H_h[b]), o["H"], ctx=f"b={b} k={k}")
                    near = abs(o["H"] - self.states[b].T_G.value) < TOL
                    rep.near_threshold += near
                    if bool(stop_h[b]) != o["stop"]:
                        if not near:
                            self._fail(f"stop flag b={b} k={k}: gpu {bool(stop_h[b])} oracle {o['stop']}"
                                       f" H={o['H']} T_G={self.states[b].T_G.value}")
                        rep.flips += 1
                        self.active[b] = 0 if o["stop"] else 1
        self.x.copy_(self.tokk.T)
        tok_h = self.tokk.cpu().numpy()
        H_h = self.Hk.cpu().numpy()
        lse_h = self.lsek.cpu().numpy()
        dl_h = self.draft_len.cpu().numpy().copy()
        stop_h_all = self.stopk.cpu().numpy()
        x_fix = {}
        for b in self.follow:
            steps = o_draft[b]
            K_t = len(steps)
            if b in skip:                       # the oracle's window and tokens are taken as they are
                self.draft_len[b] = K_t
                for k, o in enumerate(steps):
                    self.x[b, k] = o["token"]
                continue
            if dl_h[b] != K_t:
                self._fail(f"window b={b}: gpu {dl_h[b]} oracle {K_t}")
            _bump(rep.window_hist, K_t)
            for k, o in enumerate(steps):
                rep.draft_rows += 1
                self._close("H_draft", float(H_h[k, b]), o["H"], ctx=f"b={b} k={k}")
                self._close("lse_draft", float(lse_h[k, b]), o["lse"], ctx=f"b={b} k={k}")
                if not wl.adaptive_window:      # fixed window: the stop flag is still reported
                    near = abs(o["H"] - self.states[b].T_G.value) < TOL
                    rep.near_threshold += near
                    if bool(stop_h_all[k, b]) != o["stop"]:
                        if not near:
                            self._fail(f"stop flag b={b} k={k}: gpu {bool(stop_h_all[k, b])} oracle {o['stop']}")
                        rep.flips += 1
                tie = o["margin"] < TIE_EPS
                rep.near_ties += tie
                if int(tok_h[k, b]) != o["token"]:
                    if not tie:
                        self._fail(f"draft token b={b} k={k}: gpu {tok_h[k, b]} oracle {o['token']} "
                                   f"margin {o['margin']:.3e}")
                    rep.tie_flips += 1
                    x_fix[(b, k)] = o["token"]
        for (b, k), tok in x_fix.items():       # the GPU adopts the oracle's token
            self.x[b, k] = tok

        # ---- verify
        self.gs.target_rows(r, self.zt)
        dl = self.draft_len if wl.adaptive_window else None
        if wl.vanilla:
            u_vacc, u_res = U["vanilla_accept"], U["resample"]
            self.ctx.vanilla_verify(self.zd, self.zt, self.x, self._up(u_vacc), self._up(u_res),
                                    self.v_accept_len, self.v_next_token, draft_len=dl,
                                    alpha_out=self.alpha)
        self.ctx.verify(self.zd, self.zt, self.x, g_ut, g_ua, self.accept_len, self.next_token,
                        draft_len=dl, record=self.rec, fuse_update=True)
        rec = {k: v.cpu().numpy() for k, v in self.rec.items()}
        al_h = self.accept_len.cpu().numpy()
        nt_h = self.next_token.cpu().numpy()
        x_h = self.x.cpu().numpy()
        T_dev, nE_dev, nA_dev, nR_dev = (t.cpu().numpy() for t in self.ctx.get_thresholds())

        def verify_phase(n):
            b = self.follow[n]
            st = self.states[b]
            K_t = len(o_draft[b])
            LA0 = st.LA[: st.nA.value].copy()
            LR0 = st.LR[: st.nR.value].copy()
            o = oracle.verify_round(st, hd[n], ht[n], x_h[b, :K_t], u_target[b], u_accept[b], K_t=K_t)
            ov = None
            if wl.vanilla:
                ov = oracle.vanilla_round(hd[n][:K_t], ht[n], x_h[b, :K_t], u_vacc[b, :K_t], float(u_res[b]))
            return LA0, LR0, o, ov
        o_verify = list(self.pool.map(verify_phase, range(len(self.follow))))

        for n, b in enumerate(self.follow):
            st = self.states[b]
            K_t = len(o_draft[b])
            LA0, LR0, o, ov = o_verify[n]
            if b in skip:
                self._resync(b)
                continue
            rep.positions += K_t + 1
            _bump(rep.accept_hist, o["accept_len"])
            rep.n_rejections += o["rejected"]
            flagged_first = None      # first position whose decision is near its threshold
            flagged_r6 = False        # ... and it was flagged for a distance within TOL of 0 or 1
            for i in range(K_t + 1):
                c = f"b={b} i={i}"
                self._close("H_t", float(rec["H_t"][b, i]), o["H_t"][i], ctx=c)
                self._close("lse_t", float(rec["lse_t"][b, i]), o["lse_t"][i], ctx=c)
                tie = o["y_margin"][i] < TIE_EPS
                rep.near_ties += tie
                y_ok = int(rec["y"][b, i]) == int(o["y"][i])
                if not y_ok:
                    if not tie:
                        self._fail(f"target sample {c}: gpu {rec['y'][b, i]} oracle {o['y'][i]} "
                                   f"margin {o['y_margin'][i]:.3e}")
                    rep.tie_flips += 1
                    if flagged_first is None:
                        flagged_first = i
                if i == K_t:
                    break
                self._close("H_d", float(rec["H_d"][b, i]), o["H_d"][i], ctx=c)
                self._close("lse_d", float(rec["lse_d"][b, i]), o["lse_d"][i], ctx=c)
                self._close("jsd", float(rec["jsd"][b, i]), o["jsd"][i], ctx=c)
                self._close("dist", float(rec["dist"][b, i]), o["dist"][i], tol=dist_tolerance(o["dist"][i]), ctx=c)
                rep.dist_checked += 1
                rep.dist_beyond_tol += abs(float(rec["dist"][b, i]) - o["dist"][i]) > TOL
                d = o["dist"][i]
                near = (d < TOL) or (d > 1.0 - TOL)
                near_end = near
                if i <= o["accept_len"]:
                    # P(A|d) for the positions the oracle's loop reached
                    extra = [o["dist"][j] for j in range(i) if 0.0 < o["dist"][j] < 1.0]
                    LAi = np.concatenate([LA0, extra])
                    P = o["p_acc"][i]
                    Plo = oracle.accept_prob(LAi, LR0, max(d - TOL, 0.0), st.min_samples, st.bw_rule)
                    Phi = oracle.accept_prob(LAi, LR0, min(d + TOL, 1.0), st.min_samples, st.bw_rule)
                    sens = max(abs(Plo - P), abs(Phi - P))
                    self.report.err("p_acc_sensitivity", sens)
                    self._close("p_acc", float(rec["p_acc"][b, i]), P, tol=TOL + sens, ctx=c)
                    rep.p_acc_checked += 1
                    rep.p_acc_beyond_tol += abs(float(rec["p_acc"][b, i]) - P) > TOL
                    u = float(u_accept[b, i])
                    # the rejection rule in force: Bernoulli (u >= P) or the fixed threshold P < 1/2
                    cut = u if self.reject_rule == 0 else 0.5
                    decisions = {cut >= P, cut >= Plo, cut >= Phi} if self.reject_rule == 0 else \
                                {P < cut, Plo < cut, Phi < cut}
                    if x_h[b, i] != o["y"][i] and (abs(cut - P) < TOL or len(decisions) > 1):
                        near = True
                if near:
                    rep.near_threshold += 1
                    if flagged_first is None:
                        flagged_first = i
                        flagged_r6 = near_end

            # decisions
            agree = (int(al_h[b]) == o["accept_len"] and int(nt_h[b]) == o["next_token"]
                     and int(rec["rejected"][b]) == int(o["rejected"]))
            sizes_ok = (int(nE_dev[b]) == st.nE.value and int(nA_dev[b]) == st.nA.value
                        and int(nR_dev[b]) == st.nR.value)
            if not (agree and sizes_ok):
                first_diff = min(int(al_h[b]), o["accept_len"])
                if flagged_first is None or (not agree and flagged_first > first_diff):
                    self._fail(f"decision b={b}: gpu accept_len {al_h[b]} next {nt_h[b]} rejected "
                               f"{rec['rejected'][b]} sizes {(nE_dev[b], nA_dev[b], nR_dev[b])}; oracle "
                               f"accept_len {o['accept_len']} next {o['next_token']} rejected {o['rejected']} "
                               f"sizes {(st.nE.value, st.nA.value, st.nR.value)}; p_acc gpu "
                               f"{rec['p_acc'][b, :K_t]} oracle {o['p_acc']} u {u_accept[b, :K_t]}")
                rep.flips += 1
                rep.r6_resyncs += flagged_r6
                self._resync(b)
            else:
                self._close("T_G", float(T_dev[b]), st.T_G.value, ctx=f"b={b}")

            if wl.vanilla:
                _bump(rep.vanilla_accept_hist, ov["accept_len"])
                a_gpu = self.alpha[b].cpu().numpy()
                near_v = None
                for i in range(min(ov["accept_len"] + 1, K_t)):
                    self._close("alpha", float(a_gpu[i]), ov["alpha"][i], ctx=f"b={b} i={i}")
                    if abs(float(u_vacc[b, i]) - ov["alpha"][i]) < TOL:
                        rep.near_threshold += 1
                        near_v = i if near_v is None else near_v
                tie = ov["margin"] < TIE_EPS
                rep.near_ties += tie
                val, vnt = int(self.v_accept_len[b]), int(self.v_next_token[b])
                if val != ov["accept_len"]:
                    if near_v is None or near_v > min(val, ov["accept_len"]):
                        self._fail(f"vanilla accept_len b={b}: gpu {val} oracle {ov['accept_len']} "
                                   f"alpha {ov['alpha']} u {u_vacc[b, :K_t]}")
                    rep.flips += 1
                elif vnt != ov["next_token"]:
                    if not tie:
                        self._fail(f"vanilla next token b={b}: gpu {vnt} oracle {ov['next_token']} "
                                   f"margin {ov['margin']:.3e}")
                    rep.tie_flips += 1
        rep.rounds += 1
        if self.check_lists_every and rep.rounds % self.check_lists_every == 0:
            self.check_lists()

    def check_lists(self) -> None:
        """List contents on the device against the oracle's, entry by entry."""
        for b in self.follow:
            g = self.ctx.state_export(b)
            LE, LA, LR = self.states[b].lists()
            for name, a, w in (("LE", g["LE"], LE), ("LA", g["LA"], LA), ("LR", g["LR"], LR)):
                if len(a) != len(w):
                    self._fail(f"list {name} b={b}: size gpu {len(a)} oracle {len(w)}")
                if len(a):
                    diff = np.abs(a.astype(np.float64) - w)
                    e = float(diff.max())
                    self.report.err("list_" + name, e)
                    tol = TOL if name == "LE" else np.array([dist_tolerance(float(x)) for x in w])
                    if (diff > tol).any():
                        self._fail(f"list {name} b={b}: max |diff| {e:.3e}")
            self._close("T_G", g["T_G"], self.states[b].T_G.value, ctx=f"b={b} (export)")

    def run(self, rounds: Optional[int] = None) -> Report:
        for r in range(self.wl.rounds if rounds is None else rounds):
            self.round(r)
        self.check_lists()
        status = self.ctx.status()
        if status != 0:
            self._fail(f"device status word {status}")
        return self.report
