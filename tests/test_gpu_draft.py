"""GPU parity of ssd_draft_step (Algorithm 1's draft lines; Eq. 2-3) against the CPU oracle.

One draft step feeds n_in tokens at the stream's length, commits them, applies the sampling
transform to the last row and draws x ~ p.  The oracle's counterpart is its forward on the same
ids, `transform` of the last logit row and `categorical_draw` with the same uniform.  Compared per
step: the full row p (Eq. 6 consumes it later), the token, and the stream's length / pending
token.  The token is compared whenever the uniform falls inside the token's CDF interval on BOTH
sides (the oracle's row and the GPU's row) by more than 1e-5 of the mass; otherwise the rounding
of the row may have moved an edge across the uniform and the draw is skipped; so is a row whose
top-k cut keeps different ids on the two sides.
"""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth
from tests.helpers import oracle_model

pytestmark = pytest.mark.gpu

DRAW_EPS = 1e-5


def _interval(p, y):
    cdf = np.cumsum(p.astype(np.float64)) / float(np.sum(p.astype(np.float64)))
    return (float(cdf[y - 1]) if y > 0 else 0.0), float(cdf[y])


def _run(shape, lens, top_k, temperature, path, p_tol, logit_tol, seed=3):
    from paper_2505_15380_b200 import binding
    B, V = len(lens), shape.vocab_out
    wl = synth.Workload("draft", shape, shape, B, 4, temperature, top_k, tuple(lens), 2, seed, seed + 1)
    w = synth.make_weights(shape, seed)
    om = oracle_model(shape, w)
    gm = binding.Model(shape, synth.weights_blob(shape, w))
    cap = max(lens) + 16
    gs = binding.Streams(gm, B, cap, 4)
    gs.set_path(path)
    prefixes = [synth.make_prefix(wl, b) for b in range(B)]
    gs.prefill(prefixes)
    ost = []
    for b in range(B):
        st = orc.Stream(om, cap)
        orc.prefill(om, st, prefixes[b])
        ost.append(st)
    dev = gm.device
    par = binding.VerifyParams(4, temperature, top_k, 0.0)
    d_tok = torch.zeros(B, dtype=torch.int32, device=dev)
    d_p = torch.zeros((B, V), dtype=torch.float32, device=dev)
    # Algorithm 1 feeds the draft [pending], then its own tokens; after a fully accepted iteration
    # the next step feeds two ids, [x_gamma, y].  Steps: 1, 1, 1, then one with n_in = 2, then 1.
    plan = [1, 1, 1, 2, 1]
    compared = excluded = 0
    last_tok = np.array([st.pending for st in ost], dtype=np.int32)
    rng = np.random.Generator(np.random.Philox(key=seed + 50))
    for step, n_in in enumerate(plan):
        u = synth.verify_uniforms(seed + 9, B, 1, step=step)[:, 0, 1].copy()
        if n_in == 1:
            ids = last_tok.reshape(B, 1)
        else:   # [x_gamma, y]: the last drawn token and a stand-in for the verifier's new token
            ids = np.stack([last_tok, rng.integers(0, V, size=B).astype(np.int32)], axis=1)
        gs.draft_step(torch.from_numpy(np.ascontiguousarray(ids, np.int32)).to(dev), n_in,
                      torch.from_numpy(u).to(dev), par, d_tok, d_p)
        torch.cuda.synchronize()
        assert gs.last_status() == 0
        g_tok, g_p = d_tok.cpu().numpy(), d_p.cpu().numpy().astype(np.float64)
        lens_g, pend_g = gs.get_state()
        for b in range(B):
            st = ost[b]
            lg = orc.forward(om, st, ids[b])
            st.length += n_in
            p = orc.transform(lg[-1], temperature, top_k)
            same_support = np.array_equal(p > 0, g_p[b] > 0)     # same ids kept by the top-k cut
            if not same_support:      # only possible when the cut separates two nearly equal logits
                z = np.sort(lg[-1] / temperature)[::-1]
                assert 0 < top_k < V and z[top_k - 1] - z[top_k] < 1e-3, "top-k sets differ"
            else:
                assert np.abs(g_p[b] - p).max() <= p_tol, f"step {step} stream {b}: p rows differ"
            assert abs(g_p[b].sum() - 1.0) < 1e-4
            x, _ = orc.categorical_draw(p, float(u[b]))
            lo1, hi1 = _interval(p, x)
            lo2, hi2 = _interval(g_p[b], x)
            if max(lo1, lo2) + DRAW_EPS <= float(u[b]) < min(hi1, hi2) - DRAW_EPS and same_support:
                assert g_tok[b] == x, f"step {step} stream {b}: token {g_tok[b]} vs {x}"
                compared += 1
            else:
                excluded += 1
            st.pending = int(g_tok[b])                # follow the GPU's trajectory
            assert lens_g[b] == st.length and pend_g[b] == st.pending
        last_tok = g_tok.astype(np.int32).copy()
    print(f"draft steps compared {compared}, excluded {excluded}")
    assert compared >= 1 and excluded <= max(1, (compared + excluded) // 10)


@pytest.mark.parametrize("top_k,temperature", [(0, 1.0), (25, 0.8)])
def test_draft_step_fp32_tiny_draft(top_k, temperature):
    """The 1-layer fp32 draft of the tiny configuration (generic kernels)."""
    shape = synth.workload(0).draft
    _run(shape, [20, 64, 33], top_k, temperature, path=0, p_tol=1e-5, logit_tol=2e-4)


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("top_k,temperature", [(0, 1.0), (25, 0.8)])
def test_draft_step_bf16_draft_shape(path, top_k, temperature):
    """A bf16 draft with the head layout of the 4-layer draft (8/2 heads of 64), two layers deep,
    through the persistent kernel (path 0: forwards of 2-4 rows) and the generic kernels."""
    shape = synth.ModelShape(2, 256, 8, 2, 64, 512, 700, 16, 1e6)
    _run(shape, [40, 65], top_k, temperature, path=path, p_tol=1e-4, logit_tol=3e-2)
