"""Runs one verify-step workload on the CUDA path and on the oracle and compares them.

Used by the GPU parity tests and by the smoke check.  The comparison rules:

* logits: max-abs difference within `logit_tol` (3e-2 for bf16 storage, 2e-4 for fp32);
* token decisions, strict: the oracle's acceptance arithmetic applied to the GPU's own logits
  must reproduce the GPU's (k, y) exactly, except for draws closer than 1e-3 to a decision
  boundary (|r_i - a_i| < 1e-3, a categorical draw within 1e-5 (in mass) of a CDF edge, or a
  top-k cut whose neighbours differ by < 1e-5), after which the stream-step is no longer compared;
* token decisions, end to end: the pure oracle's (k, y) must equal the GPU's unless r_i falls
  between the two sides' thresholds (widened by 1e-3), or the draw's uniform falls within 1e-5
  (in mass) of where either side puts a CDF edge of the oracle's token, or the two sides keep
  different top-k sets, i.e. unless the logit rounding moved a boundary across the uniform or an
  id across the cut.  A bare disagreement is a failure.

Excluded stream-steps are counted and bounded: a case passes only if at least one decision was
compared and the excluded share stays small.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import numpy as np
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import binding, synth
from tests.helpers import crafted_draft_rows, oracle_model

WINDOW = 1e-3        # acceptance test: |a_i - r_i| closer than this is not compared
# Categorical draws and top-k cuts.  The strict comparison applies the oracle's float64 arithmetic
# to the GPU's own logits, so the two sides differ only by fp32 rounding of exp, of the row sum and
# of logit / T (about 1e-6 of the total mass, 1e-7 relative in z): a draw is skipped when it lies
# within 1e-5 (in mass) of a CDF edge, a top-k cut when its two neighbours differ by < 1e-5.
# End to end both CDFs are built explicitly and the uniform must fall inside the token's interval
# on both sides by 1e-5; a top-k row is skipped only if the two sides really keep different sets.
DRAW_WINDOW = 1e-5
DRAW_EPS = 1e-5
TOPK_GAP = 1e-5


@dataclasses.dataclass
class CaseResult:
    max_logit_err: float
    n_streams: int
    n_strict_excluded: int
    n_e2e_excluded: int
    ks: List[int]


def synthetic_kv(streams: binding.Streams, lens, seed: int, std: float = 0.6) -> None:
    synth.fill_synthetic_kv(streams.kv, lens, seed, std)


def oracle_stream_from_gpu_kv(model: orc.Model, streams: binding.Streams, b: int, n: int,
                              pending: int) -> orc.Stream:
    st = orc.Stream(model, streams.capacity)
    kv = streams.kv[:, b, :, :, :n, :].to(torch.float32).cpu().numpy().astype(np.float64)
    for l in range(model.L):
        st.K[l][:n] = kv[l, 0].transpose(1, 0, 2)
        st.V[l][:n] = kv[l, 1].transpose(1, 0, 2)
    st.length, st.pending = n, pending
    return st


def _topk_gap_small(logits_row: np.ndarray, temperature: float, top_k: int) -> bool:
    V = logits_row.shape[0]
    if not (0 < top_k < V):
        return False
    z = np.sort(logits_row / temperature)[::-1]
    return bool(z[top_k - 1] - z[top_k] < TOPK_GAP)


def _nucleus_edge_close(logits_row: np.ndarray, temperature: float, top_k: int, top_p: float) -> bool:
    """True when the running mass at the nucleus cut lies within 1e-5 of top_p: fp32 rounding of
    the masses may then move the cut by one id."""
    if not (0.0 < top_p < 1.0):
        return False
    full = np.sort(orc.transform(logits_row, temperature, top_k))[::-1]
    cum = np.cumsum(full)
    return bool(np.min(np.abs(cum - top_p)) < 1e-5)


def _draw_interval(q_row: np.ndarray, p_row: Optional[np.ndarray], y: int):
    """[lo, hi) of token y in the normalised CDF the new token is drawn from: the residual
    max(0, q - p) after a rejection (q itself when that has no mass), q for the bonus token."""
    w = q_row.astype(np.float64)
    if p_row is not None:
        r = np.maximum(0.0, w - p_row.astype(np.float64))
        w = r if r.sum() > 0.0 else w
    cdf = np.cumsum(w) / w.sum()
    return (float(cdf[y - 1]) if y > 0 else 0.0), float(cdf[y])


def check_exclusions(res: "CaseResult", max_strict_frac: float = 0.10,
                     max_e2e_frac: float = 0.34) -> None:
    """A parity case must have compared something, and may skip only a small share."""
    n = res.n_streams
    assert n >= 1 and n - res.n_strict_excluded >= 1, "no decision was compared"
    assert res.n_strict_excluded <= max(1, int(np.ceil(max_strict_frac * n))), \
        f"{res.n_strict_excluded} of {n} stream-steps excluded from the strict comparison"
    assert res.n_e2e_excluded <= max(1, int(np.ceil(max_e2e_frac * n))), \
        f"{res.n_e2e_excluded} of {n} stream-steps excluded from the end-to-end comparison"


def run_case(wl: synth.Workload, *, beta: float, sigma: float, kv_mode: str = "prefill",
             oracle_streams: Optional[List[int]] = None, logit_tol: Optional[float] = None,
             uniform_seed: int = 0, commit_and_repeat: bool = False,
             capacity: Optional[int] = None, path: int = 0, split: bool = True,
             max_strict_frac: float = 0.10, max_e2e_frac: float = 0.34, top_p: float = 0.0,
             paged: Optional[tuple] = None, ras: Optional[tuple] = None,
             attn_kernel: int = 0) -> CaseResult:
    """kv_mode 'prefill': both sides load the seeded prefix through their own forward;
    'synthetic': seeded random K/V is written to the cache and handed to the oracle as input."""
    shape = wl.target
    B, gamma, R, V = wl.batch, wl.gamma, wl.gamma + 1, shape.vocab_out
    if logit_tol is None:
        logit_tol = 2e-4 if shape.weight_dtype == synth.F32 else 3e-2
    w = synth.make_weights(shape, wl.model_seed)
    omodel = oracle_model(shape, w)
    gmodel = binding.Model(shape, synth.weights_blob(shape, w))
    cap = capacity or (max(wl.prefix_lens) + 2 * R + 8)
    if paged:          # (pages in the pool, pages per stream): K/V in 64-token pages
        gs = binding.PagedStreams(gmodel, B, paged[0], paged[1], gamma)
        cap = gs.capacity
    else:
        gs = binding.Streams(gmodel, B, cap, gamma)
    gs.set_path(path)          # 0: persistent kernel where the forward fits it, 1: generic kernels
    gs.set_attention_kernel(attn_kernel)   # batched forward: 0 by key range, 1 warp-level, 2 tcgen05
    gs.set_activation_split(split)   # persistent kernel: bf16 activations, or bf16 hi + lo pairs
    which = list(range(B)) if oracle_streams is None else list(oracle_streams)
    prefixes = [synth.make_prefix(wl, b) for b in range(B)]
    ostreams = {}
    if kv_mode == "prefill":
        gs.prefill(prefixes)
        for b in which:
            st = orc.Stream(omodel, cap)
            orc.prefill(omodel, st, prefixes[b])
            ostreams[b] = st
    else:
        lens = [len(p) - 1 for p in prefixes]
        synthetic_kv(gs, lens, seed=wl.data_seed + 100)
        gs.kv_truncate(lens, [int(p[-1]) for p in prefixes])
        for b in which:
            ostreams[b] = oracle_stream_from_gpu_kv(omodel, gs, b, lens[b], int(prefixes[b][-1]))
    lens_g, pend_g = gs.get_state()
    for b in which:
        assert lens_g[b] == ostreams[b].length and pend_g[b] == ostreams[b].pending

    # repetition-aware sampling (window, tau): the last `window` tokens of each T_in, pending last
    win, tau = ras if ras else (0, 0.0)
    recent = np.full((B, max(win, 1)), -1, dtype=np.int32)
    for b in range(B):
        tail = prefixes[b][-win:] if win else prefixes[b][:0]
        if win:
            recent[b, win - len(tail):] = tail
    n_ras_active = 0
    n_steps = 2 if commit_and_repeat else 1
    res = CaseResult(0.0, 0, 0, 0, [])
    dev = gmodel.device
    for step in range(n_steps):
        uni = synth.verify_uniforms(uniform_seed, B, R, step=step)
        # ---- draft rows: crafted from sequential ORACLE decodes for the checked streams,
        #      generic random rows elsewhere
        p_rows = synth.random_prob_rows(B * gamma, V, seed=wl.data_seed + step, support=64
                                        ).reshape(B, gamma, V)
        draft = synth.sample_from_rows(p_rows.reshape(-1, V), seed=wl.data_seed + 5 + step
                                       ).reshape(B, gamma)
        for b in which:
            st = ostreams[b]
            base_len = st.length
            tok = st.pending
            for i in range(gamma):
                lg = orc.forward(omodel, st, np.array([tok]))[0]
                st.length += 1
                row = crafted_draft_rows(lg[None], sigma, wl.temperature, wl.top_k,
                                         seed=1000 * b + 10 * i + step)[0]
                p_rows[b, i] = row
                tok = int(synth.sample_from_rows(row[None], seed=77 + 1000 * b + i + step)[0])
                draft[b, i] = tok
            st.length = base_len
        # ---- GPU
        d_recent = torch.from_numpy(recent).to(dev)
        params = binding.VerifyParams(gamma, wl.temperature, wl.top_k, beta, top_p, win, tau,
                                      d_recent.data_ptr() if win else None)
        d_tok = torch.from_numpy(draft.astype(np.int32)).to(dev)
        d_p = torch.from_numpy(p_rows.astype(np.float32)).to(dev)
        d_u = torch.from_numpy(uni).to(dev)
        d_k = torch.zeros(B, dtype=torch.int32, device=dev)
        d_y = torch.zeros(B, dtype=torch.int32, device=dev)
        d_logits = torch.zeros((B, R, V), dtype=torch.float32, device=dev)
        gs.verify(d_tok, d_p, d_u, params, d_k, d_y, d_logits)
        torch.cuda.synchronize()
        assert gs.last_status() == 0
        # same call again without a commit: must be bit-identical (no races, no stale state)
        d_k2, d_y2, d_l2 = torch.zeros_like(d_k), torch.zeros_like(d_y), torch.zeros_like(d_logits)
        gs.verify(d_tok, d_p, d_u, params, d_k2, d_y2, d_l2)
        torch.cuda.synchronize()
        assert torch.equal(d_k, d_k2) and torch.equal(d_y, d_y2) and torch.equal(d_logits, d_l2)
        g_k, g_y, g_logits = d_k.cpu().numpy(), d_y.cpu().numpy(), d_logits.cpu().numpy()
        assert ((g_k >= 0) & (g_k <= gamma)).all() and ((g_y >= 0) & (g_y < V)).all()
        # ---- oracle and comparison
        for b in which:
            st = ostreams[b]
            o = orc.verify(omodel, st, draft[b], p_rows[b], uni[b], temperature=wl.temperature,
                           top_k=wl.top_k, beta=beta, top_p=top_p, recent=recent[b], win_size=win, tau_r=tau)
            err = float(np.abs(o["logits"] - g_logits[b]).max())
            res.max_logit_err = max(res.max_logit_err, err)
            assert err <= logit_tol, f"stream {b}: logits differ by {err}"
            # strict: oracle arithmetic on the GPU's logits
            gl = g_logits[b].astype(np.float64)
            if win:
                hist = np.concatenate([recent[b].astype(np.int64), draft[b].astype(np.int64)])
                q_g = np.stack([orc.transform_ras(r, wl.temperature, wl.top_k, top_p, hist[:win + i], win, tau)
                                for i, r in enumerate(gl)])
                n_ras_active += int(any(not np.allclose(q_g[i], orc.transform(gl[i], wl.temperature, wl.top_k, top_p))
                                        for i in range(R)))
            else:
                q_g = np.stack([orc.transform(r, wl.temperature, wl.top_k, top_p) for r in gl])
            o2 = orc.accept_step(q_g, p_rows[b], draft[b], uni[b], beta)
            res.n_streams += 1
            res.ks.append(int(g_k[b]))
            strict_excl = False
            n_eval = min(o2["k"] + 1, gamma)
            for i in range(n_eval):
                if abs(o2["thresholds"][i] - float(uni[b, i, 0])) < WINDOW or \
                        _topk_gap_small(gl[i], wl.temperature, wl.top_k) or \
                        _nucleus_edge_close(gl[i], wl.temperature, wl.top_k, top_p):
                    strict_excl = True
                    break
            if not strict_excl:
                assert g_k[b] == o2["k"], f"stream {b}: accepted length {g_k[b]} vs {o2['k']}"
                if o2["draw_margin"] < DRAW_WINDOW or \
                        _topk_gap_small(gl[o2["k"]], wl.temperature, wl.top_k) or \
                        _nucleus_edge_close(gl[o2["k"]], wl.temperature, wl.top_k, top_p):
                    strict_excl = True
                else:
                    assert g_y[b] == o2["y"], f"stream {b}: token {g_y[b]} vs {o2['y']}"
            res.n_strict_excluded += int(strict_excl)
            # end to end: pure oracle
            e2e_excl = False
            n_rows_eval = min(max(o["k"], o2["k"]) + 1, R)
            for i in range(n_rows_eval):
                if not np.array_equal(o["q_rows"][i] > 0, q_g[i] > 0):
                    e2e_excl = True     # the logit rounding moved an id across the top-k cut
            for i in range(min(max(o["k"], o2["k"]) + 1, gamma)):
                lo = min(o["thresholds"][i] if i < len(o["thresholds"]) else 9.0,
                         o2["thresholds"][i] if i < len(o2["thresholds"]) else 9.0) - WINDOW
                hi = max(o["thresholds"][i] if i < len(o["thresholds"]) else -9.0,
                         o2["thresholds"][i] if i < len(o2["thresholds"]) else -9.0) + WINDOW
                if lo <= float(uni[b, i, 0]) <= hi:
                    e2e_excl = True
            if not e2e_excl:
                assert g_k[b] == o["k"], f"stream {b}: e2e accepted length {g_k[b]} vs {o['k']}"
                kk = o["k"]
                prow = p_rows[b][kk] if kk < gamma else None
                lo1, hi1 = _draw_interval(o["q_rows"][kk], prow, o["y"])
                lo2, hi2 = _draw_interval(q_g[kk], prow, o["y"])
                ud = float(uni[b, kk, 1])
                if max(lo1, lo2) + DRAW_EPS <= ud < min(hi1, hi2) - DRAW_EPS:
                    assert g_y[b] == o["y"], f"stream {b}: e2e token {g_y[b]} vs {o['y']}"
                else:
                    e2e_excl = True       # the uniform sits at an edge one side may have moved
            res.n_e2e_excluded += int(e2e_excl)
            if commit_and_repeat:
                orc.commit(st, int(g_k[b]), int(g_y[b]))      # follow the GPU's trajectory
                if win:
                    emitted = np.concatenate([draft[b][:int(g_k[b])], [int(g_y[b])]]).astype(np.int32)
                    recent[b] = np.concatenate([recent[b], emitted])[-win:]
        if commit_and_repeat:
            gs.kv_commit(d_k, d_y)
            torch.cuda.synchronize()
            lens_g, pend_g = gs.get_state()
            for b in which:
                assert lens_g[b] == ostreams[b].length and pend_g[b] == ostreams[b].pending
    print(f"[{wl.name}] streams-steps {res.n_streams}, strict excluded {res.n_strict_excluded}, "
          f"e2e excluded {res.n_e2e_excluded}, max|dlogit| {res.max_logit_err:.2e}, k {res.ks}")
    check_exclusions(res, max_strict_frac, max_e2e_frac)
    if win:
        assert n_ras_active >= 1, "no row had a repeated id in its window: the case does not test the mixture"
    return res
