"""ssd_accept_noalloc against ssd_verify (collected last on purpose: see the file name).

ssd_accept_noalloc serves callers that may not allocate device memory - a serving loop with a
memory pool fixed at start-up, or a plug-in that only receives device pointers - by keeping the
acceptance kernel's scratch in a fixed array inside the library.  It must return exactly what
ssd_verify returns for the same logits, also on a second call, which finds the shared array as
the first call left it.
"""
import numpy as np
import pytest
import torch

from paper_2505_15380_b200 import synth

pytestmark = pytest.mark.gpu


def test_accept_noalloc_matches_verify_on_two_calls_in_a_row():
    from paper_2505_15380_b200 import binding
    shape = synth.ModelShape(2, 128, 4, 2, 64, 256, 700, 8, 1e6)
    B, gamma, V = 5, 4, shape.vocab_out
    wl = synth.Workload("noalloc", shape, shape, B, gamma, 0.8, 25, (30, 64, 65, 9, 120), 2, 41, 42)
    model = binding.Model(shape, synth.weights_blob(shape, synth.make_weights(shape, 41)))
    gs = binding.Streams(model, B, 160, gamma)
    gs.prefill([synth.make_prefix(wl, b) for b in range(B)])
    dev = model.device
    calls = []
    for call, (beta, top_k, temperature) in enumerate([(0.0, 25, 0.8), (0.4, 0, 1.0)]):
        p = synth.random_prob_rows(B * gamma, V, seed=call, sharpness=1.0).reshape(B, gamma, V)
        x = synth.sample_from_rows(p.reshape(-1, V), seed=10 + call).reshape(B, gamma)
        u = synth.verify_uniforms(5, B, gamma + 1, step=call)
        par = binding.VerifyParams(gamma, temperature, top_k, beta)
        d_x = torch.from_numpy(x.astype(np.int32)).to(dev)
        d_p = torch.from_numpy(p).to(dev)
        d_u = torch.from_numpy(u).to(dev)
        k_ref = torch.full((B,), -1, dtype=torch.int32, device=dev)
        y_ref = torch.full((B,), -1, dtype=torch.int32, device=dev)
        logits = torch.zeros((B, gamma + 1, V), dtype=torch.float32, device=dev)
        gs.verify(d_x, d_p, d_u, par, k_ref, y_ref, logits)       # existing entry point
        torch.cuda.synchronize()
        calls.append((par, d_x, d_p, d_u, logits, k_ref, y_ref))
    results = []
    for par, d_x, d_p, d_u, logits, k_ref, y_ref in calls:        # two no-alloc calls in a row
        k = torch.full((B,), -2, dtype=torch.int32, device=dev)
        y = torch.full((B,), -2, dtype=torch.int32, device=dev)
        binding.accept_noalloc(logits, d_x, d_p, d_u, par, k, y)
        results.append((k, y))
    torch.cuda.synchronize()
    from oracle import ssd_oracle as orc
    compared = 0
    for (k, y), (par, d_x, d_p, d_u, logits, k_ref, y_ref) in zip(results, calls):
        # same kernel, same inputs: integer outputs must agree exactly
        assert torch.equal(k, k_ref) and torch.equal(y, y_ref)
        # and both must be what the oracle's acceptance step makes of these logits (decisions
        # closer than 1e-3 to a boundary are not compared)
        lg, xs, ps, us = (t.cpu().numpy() for t in (logits, d_x, d_p, d_u))
        for b in range(B):
            q = np.stack([orc.transform(r.astype(np.float64), par.temperature, par.top_k) for r in lg[b]])
            o = orc.accept_step(q, ps[b], xs[b], us[b], par.beta)
            near = any(abs(a - float(us[b, i, 0])) < 1e-3 for i, a in enumerate(o["thresholds"]))
            zs = np.sort(lg[b] / par.temperature, axis=1)[:, ::-1]
            if 0 < par.top_k < V and (zs[:, par.top_k - 1] - zs[:, par.top_k]).min() < 1e-5:
                near = True
            if near:
                continue
            assert int(k[b]) == o["k"]
            if o["draw_margin"] >= 1e-5:      # same logits on both sides: only fp32 rounding differs
                assert int(y[b]) == o["y"]
                compared += 1
    assert compared >= B      # at least half of the 2 x B stream-steps were checked to the token


def test_accept_noalloc_rejects_an_impossible_draft_token():
    """This call has no status word to report through, so a draft token outside the vocabulary
    (or a draft probability that is not one) must end the accepted prefix in front of it."""
    from paper_2505_15380_b200 import binding
    dev = torch.device("cuda:0")
    B, gamma, V = 2, 4, 300
    p = synth.random_prob_rows(B * gamma, V, seed=3, sharpness=0.5).reshape(B, gamma, V)
    logits = torch.from_numpy(np.log(p[:, [0, 1, 2, 3, 3]]).astype(np.float32)).to(dev).contiguous()  # q_i = p_i
    x = synth.sample_from_rows(p.reshape(-1, V), seed=4).reshape(B, gamma).astype(np.int32)
    u = synth.verify_uniforms(6, B, gamma + 1)
    par = binding.VerifyParams(gamma, 1.0, 0, 0.0)
    k = torch.full((B,), -2, dtype=torch.int32, device=dev)
    y = torch.full((B,), -2, dtype=torch.int32, device=dev)
    args = (torch.from_numpy(p).to(dev), torch.from_numpy(u).to(dev), par, k, y)
    binding.accept_noalloc(logits, torch.from_numpy(x).to(dev), *args)
    torch.cuda.synchronize()
    assert k.tolist() == [gamma, gamma]            # p = q: everything is accepted
    x[0, 2] = V + 5                                # impossible token at position 3 of stream 0
    p_bad = p.copy()
    p_bad[1, 1, x[1, 1]] = np.nan                  # impossible probability at position 2 of stream 1
    binding.accept_noalloc(logits, torch.from_numpy(x).to(dev), torch.from_numpy(p_bad).to(dev),
                           torch.from_numpy(u).to(dev), par, k, y)
    torch.cuda.synchronize()
    assert k.tolist() == [2, 1]
    assert 0 <= int(y[0]) < V and 0 <= int(y[1]) < V


def test_accept_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2505_15380_b200 import binding
    L = binding.lib()
    dev = torch.device("cuda:0")
    buf = torch.zeros(1024, dtype=torch.float32, device=dev)
    out = torch.zeros(512, dtype=torch.int32, device=dev)
    par = binding.VerifyParams(4, 1.0, 0, 0.0)
    import ctypes
    args = (buf.data_ptr(), out.data_ptr(), buf.data_ptr(), buf.data_ptr(), ctypes.byref(par))
    assert L.ssd_accept_noalloc(*args, 257, 16, out.data_ptr(), out.data_ptr(), None) == -6
    big = binding.VerifyParams(16, 1.0, 0, 0.0)
    assert L.ssd_accept_noalloc(buf.data_ptr(), out.data_ptr(), buf.data_ptr(), buf.data_ptr(),
                                ctypes.byref(big), 1, 16, out.data_ptr(), out.data_ptr(), None) == -3
    assert L.ssd_accept_noalloc(None, out.data_ptr(), buf.data_ptr(), buf.data_ptr(),
                                ctypes.byref(par), 1, 16, out.data_ptr(), out.data_ptr(), None) == -1
