"""Algorithm 1 end to end on the GPU (ssd_iteration: draft x gamma, verify, accept, both commits,
emitted tokens; no host decision inside an iteration) against the same loop on the CPU oracle.

The GPU loop is run one iteration at a time so that every iteration's draft tokens, draft rows,
accepted length and new token can be read back; the oracle recomputes each of them from its own
state and then follows the GPU's choice, so that one knife-edge draw cannot derail the rest of the
comparison.  A second test replays the captured iteration as a CUDA graph and checks that the
device-resident loop emits exactly what the step-by-step loop emitted.
"""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth
from tests.helpers import oracle_model

pytestmark = pytest.mark.gpu

WINDOW = 1e-3


def _interval(w, y):
    w = np.asarray(w, np.float64)
    cdf = np.cumsum(w) / w.sum()
    return (float(cdf[y - 1]) if y > 0 else 0.0), float(cdf[y])


def _pool(seed, n_iter, B, gamma):
    per = gamma + 2 * (gamma + 1)
    return np.stack([synth.verify_uniforms(seed, B, per, step=it)[:, :, 0] for it in range(n_iter)]
                    ).astype(np.float32)


def _setup(tshape, dshape, lens, gamma, seed, n_iter, out_cap=256, ras_window=0):
    from paper_2505_15380_b200 import binding
    B = len(lens)
    wl = synth.Workload("loop", tshape, dshape, B, gamma, 1.0, 0, tuple(lens), 2, seed, seed + 1)
    tw, dw = synth.make_weights(tshape, seed), synth.make_weights(dshape, seed + 7)
    tm = binding.Model(tshape, synth.weights_blob(tshape, tw))
    dm = binding.Model(dshape, synth.weights_blob(dshape, dw))
    cap = max(lens) + n_iter * (gamma + 1) + gamma + 8
    ts, ds = binding.Streams(tm, B, cap, gamma), binding.Streams(dm, B, cap, max(gamma, 1))
    prefixes = [synth.make_prefix(wl, b) for b in range(B)]
    ts.prefill(prefixes)
    ds.prefill(prefixes)
    pool = _pool(seed + 3, n_iter, B, gamma)
    loop = binding.Loop(ts, ds, prefixes, gamma, pool, out_cap, ras_window=ras_window)
    return tm, dm, ts, ds, prefixes, pool, loop, tw, dw, cap


def _run_against_oracle(tshape, dshape, lens, gamma, temperature, top_k, beta, n_iter, p_tol, draw_eps,
                        seed=5, ras=None):
    from paper_2505_15380_b200 import binding
    win, tau = ras if ras else (0, 0.0)
    tm, dm, ts, ds, prefixes, pool, loop, tw, dw, cap = _setup(tshape, dshape, lens, gamma, seed, n_iter,
                                                               ras_window=win)
    B, V = len(lens), tshape.vocab_out
    otm, odm = oracle_model(tshape, tw), oracle_model(dshape, dw)
    ot, od, in_ids = [], [], []
    for b in range(B):
        st, sd = orc.Stream(otm, cap), orc.Stream(odm, cap)
        orc.prefill(otm, st, prefixes[b])
        orc.prefill(odm, sd, prefixes[b])
        sd.length -= 1                                   # the draft re-feeds the last two ids
        ot.append(st)
        od.append(sd)
        in_ids.append([int(prefixes[b][-2]), int(prefixes[b][-1])])
    par = binding.VerifyParams(gamma, temperature, top_k, beta, 0.0, win, tau,
                               loop.recent.data_ptr() if win else None)
    recent = loop.recent.cpu().numpy().copy() if win else None
    emitted = [[] for _ in range(B)]
    n_dec = n_excl = 0
    seen_k = set()
    for it in range(n_iter):
        loop.iterate(par)
        torch.cuda.synchronize()
        assert ts.last_status() == 0 and ds.last_status() == 0
        g_x = loop.draft_tokens.cpu().numpy()
        g_p = loop.draft_probs.cpu().numpy()
        g_k = loop.accepted_len.cpu().numpy()
        g_y = loop.next_token.cpu().numpy()
        assert int(loop.iteration[0]) == it + 1
        tl, tp = ts.get_state()
        dl, dp = ds.get_state()
        for b in range(B):
            u = pool[it, b]
            st, sd = ot[b], od[b]
            # ---- draft: x_i ~ p_i = M_p(T_in, x_1..x_{i-1})  (Eq. 2-3)
            ids = np.array(in_ids[b])
            excl = False
            for i in range(gamma):
                lg = orc.forward(odm, sd, ids)
                sd.length += len(ids)
                p = orc.transform(lg[-1], temperature, top_k)
                same_support = np.array_equal(p > 0, g_p[b, i] > 0)
                if not same_support:
                    # the two sides keep different ids only when the top-k cut falls between two
                    # logits closer than the logit tolerance; then the rows are not comparable
                    z = np.sort(lg[-1] / temperature)[::-1]
                    assert 0 < top_k < V and z[top_k - 1] - z[top_k] < 1e-3, "top-k sets differ"
                    excl = True
                else:
                    assert np.abs(g_p[b, i] - p).max() <= p_tol, f"iteration {it} stream {b} step {i}: p rows"
                x, _ = orc.categorical_draw(p, float(u[i]))
                lo1, hi1 = _interval(p, x)
                lo2, hi2 = _interval(g_p[b, i], x)
                if same_support and max(lo1, lo2) + 1e-5 <= float(u[i]) < min(hi1, hi2) - 1e-5:
                    assert g_x[b, i] == x, f"iteration {it} stream {b}: draft token {i}"
                else:
                    excl = True
                ids = np.array([g_x[b, i]])               # follow the GPU
            # ---- verify and accept (Eq. 4-6) with the GPU's draft as input on both sides
            uni = u[gamma:].reshape(gamma + 1, 2)
            o = orc.verify(otm, st, g_x[b], g_p[b], uni, temperature=temperature, top_k=top_k, beta=beta,
                           recent=recent[b] if win else None, win_size=win, tau_r=tau)
            near = any(abs(a - float(uni[i, 0])) < WINDOW for i, a in enumerate(o["thresholds"]))
            if not near:
                assert g_k[b] == o["k"], f"iteration {it} stream {b}: accepted length"
                kk = o["k"]
                w = o["q_rows"][kk] if kk == gamma else np.maximum(0.0, o["q_rows"][kk] - g_p[b, kk])
                if w.sum() <= 0:
                    w = o["q_rows"][kk]
                lo, hi = _interval(w, o["y"])
                if lo + draw_eps <= float(uni[kk, 1]) < hi - draw_eps:
                    assert g_y[b] == o["y"], f"iteration {it} stream {b}: new token"
                else:
                    excl = True
            else:
                excl = True
            n_dec += 1
            n_excl += int(excl)
            seen_k.add(int(g_k[b]))
            # ---- append to T_in on both models, as the GPU decided
            k, y = int(g_k[b]), int(g_y[b])
            orc.commit(st, k, y)
            prev = int(g_x[b, k - 1]) if k > 0 else in_ids[b][1]
            sd.length -= gamma - k
            sd.pending = y
            in_ids[b] = [prev, y]
            emitted[b] += [int(t) for t in g_x[b, :k]] + [y]
            if win:
                recent[b] = np.concatenate([recent[b], np.array(emitted[b][-(k + 1):], np.int32)])[-win:]
            assert tl[b] == st.length and tp[b] == st.pending
            assert dl[b] == sd.length and dp[b] == y
            assert tl[b] == dl[b] + 1                    # the draft stays one token behind
    if win:
        assert np.array_equal(loop.recent.cpu().numpy(), recent)     # the device kept the window up to date
    out = loop.out_tokens.cpu().numpy()
    cnt = loop.out_count.cpu().numpy()
    assert np.array_equal(loop.in_ids.cpu().numpy(), np.array(in_ids))
    for b in range(B):
        assert cnt[b] == len(emitted[b])                 # L_acc += k + 1 per iteration
        assert out[b, :cnt[b]].tolist() == emitted[b]
    log = loop.accept_log.cpu().numpy()
    assert (log[:n_iter] >= 0).all() and int(log[:n_iter].sum()) + n_iter * B == int(cnt.sum())
    print(f"loop: {n_dec} stream-iterations, {n_excl} with a skipped decision, k seen {sorted(seen_k)}")
    assert n_excl <= max(2, n_dec // 5)
    return seen_k


def test_loop_fp32_tiny_models_25_iterations():
    """The tiny configuration's target and draft, two streams, beta = 0.4 (the paper's value)."""
    wl = synth.workload(0)
    seen = _run_against_oracle(wl.target, wl.draft, [64, 33], 4, 1.0, 0, 0.4, 25, p_tol=1e-5, draw_eps=1e-5)
    assert len(seen) >= 3


def test_loop_fp32_tiny_models_lossless_rule():
    wl = synth.workload(0)
    _run_against_oracle(wl.target, wl.draft, [20], 3, 1.0, 0, 0.0, 20, p_tol=1e-5, draw_eps=1e-5, seed=9)


def test_loop_bf16_models_top_k():
    """bf16 target and draft through the persistent kernel (verify 5 rows, draft steps 2 and 1 rows)."""
    t = synth.ModelShape(3, 256, 8, 2, 64, 512, 700, 16, 1e6)
    d = synth.ModelShape(1, 128, 4, 2, 32, 256, 700, 16, 1e6)
    _run_against_oracle(t, d, [40, 65, 17], 4, 0.8, 25, 0.4, 20, p_tol=2e-4, draw_eps=1e-3)


def test_loop_with_repetition_aware_target_sampling():
    """The window of recent tokens is kept on the device across iterations (60-id vocabulary, so
    repeats do occur)."""
    t = synth.ModelShape(2, 128, 4, 2, 64, 256, 60, 16, 1e6)
    d = synth.ModelShape(1, 128, 4, 2, 32, 256, 60, 16, 1e6)
    _run_against_oracle(t, d, [40, 21], 3, 0.9, 20, 0.4, 15, p_tol=2e-4, draw_eps=1e-3, ras=(8, 0.25))


def test_loop_batched_streams_take_the_tensor_core_path():
    """Five streams x (gamma + 1 = 5) rows = 25 verify rows: the target's forward runs on the
    tcgen05 projections; the draft's two-row first step (10 rows) on the persistent kernel."""
    t = synth.ModelShape(2, 128, 4, 2, 64, 256, 300, 16, 1e6)
    d = synth.ModelShape(1, 128, 4, 2, 32, 256, 300, 16, 1e6)
    _run_against_oracle(t, d, [30, 64, 65, 9, 120], 4, 0.8, 25, 0.4, 12, p_tol=2e-4, draw_eps=1e-3)


def test_graph_replay_of_the_iteration_equals_the_step_by_step_loop():
    """The device-resident loop: one captured iteration replayed n times, no host work in between."""
    from paper_2505_15380_b200 import binding
    t = synth.ModelShape(2, 256, 8, 2, 64, 512, 700, 16, 1e6)
    d = synth.ModelShape(1, 128, 4, 2, 32, 256, 700, 16, 1e6)
    n_iter, gamma = 30, 4
    par = binding.VerifyParams(gamma, 0.8, 25, 0.4)
    results = []
    for mode in ("steps", "graph"):
        tm, dm, ts, ds, prefixes, pool, loop, *_ = _setup(t, d, [50, 21], gamma, 13, n_iter)
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            if mode == "steps":
                for _ in range(n_iter):
                    loop.iterate(par, stream=stream)
            else:
                loop.iterate(par, stream=stream)          # sets kernel attributes outside the capture
                stream.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    loop.iterate(par, stream=stream)
                for _ in range(n_iter - 1):
                    g.replay()
            stream.synchronize()
        torch.cuda.synchronize()
        assert ts.last_status() == 0 and ds.last_status() == 0
        results.append((loop.out_tokens.cpu(), loop.out_count.cpu(), loop.accept_log.cpu(),
                        ts.get_state(), ds.get_state(), int(loop.iteration[0])))
    a, b = results
    assert a[5] == b[5] == n_iter
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2])
    assert all(np.array_equal(x, y) for x, y in zip(a[3] + a[4], b[3] + b[4]))
    assert int(a[1].min()) >= n_iter                     # every iteration emits at least one token
