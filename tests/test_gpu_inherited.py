"""A draft model made of the target's own layers (Sec. 2.3: the draft inherits layers of the
target - lower two and upper six of 24 in the paper's experiments): on the GPU the inherited
model aliases the target's weights; the oracle gets a model whose layer i simply holds the
tensors of the mapped target layer.  Compared on all three forward paths."""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth
from tests.helpers import oracle_model

pytestmark = pytest.mark.gpu


def _mapped_weights(w, layer_map):
    out = {k: v for k, v in w.items() if not k.startswith("l")}
    out["embed"] = w["embed"]
    for i, src in enumerate(layer_map):
        for k, v in w.items():
            if k.startswith(f"l{src}."):
                out[f"l{i}." + k.split(".", 1)[1]] = v
    return out


@pytest.mark.parametrize("path,batch", [(0, 1), (0, 3), (1, 2), (0, 5)])
def test_inherited_model_forward_matches_oracle(path, batch):
    """batch 1 and 3: persistent kernel (5 and 15 rows) walking the packed streams in map order;
    path 1: generic kernels; batch 5: 25 rows on the tensor-core path."""
    from paper_2505_15380_b200 import binding
    import dataclasses
    shape = synth.ModelShape(6, 128, 4, 2, 64, 256, 300, 8, 1e4)
    layer_map = [0, 1, 4, 5]
    w = synth.make_weights(shape, 17)
    for l in range(shape.n_layers):            # distinct gains, so that a wrong layer's norm shows
        w[f"l{l}.norm1"] = synth.bf16_round((1.0 + 0.1 * l + 0.01 * np.arange(128)).astype(np.float32))
        w[f"l{l}.norm2"] = synth.bf16_round((0.9 + 0.05 * l + 0.01 * np.arange(128)).astype(np.float32))
    source = binding.Model(shape, synth.weights_blob(shape, w))
    draft = binding.InheritedModel(source, layer_map)
    dshape = dataclasses.replace(shape, n_layers=len(layer_map))
    om = oracle_model(dshape, _mapped_weights(w, layer_map))
    gamma, V = 4, shape.vocab_out
    lens = [40, 65, 130, 7, 90][:batch]
    wl = synth.Workload("inh", dshape, dshape, batch, gamma, 1.0, 0, tuple(lens), 2, 3, 4)
    gs = binding.Streams(draft, batch, 160, gamma)
    gs.set_path(path)
    prefixes = [synth.make_prefix(wl, b) for b in range(batch)]
    gs.prefill(prefixes)
    dev = source.device
    x = np.random.default_rng(2).integers(0, V, size=(batch, gamma)).astype(np.int32)
    lg = torch.zeros((batch, gamma + 1, V), dtype=torch.float32, device=dev)
    gs.forward(torch.from_numpy(x).to(dev), gamma, lg)
    torch.cuda.synchronize()
    assert gs.last_status() == 0
    for b in range(batch):
        st = orc.Stream(om, 160)
        orc.prefill(om, st, prefixes[b])
        ol = orc.forward(om, st, np.concatenate([[st.pending], x[b]]))
        assert np.abs(lg[b].cpu().numpy() - ol).max() < 5e-4, (path, b)
    # the source model itself is untouched by the draft's existence
    gs2 = binding.Streams(source, 1, 160, gamma)
    gs2.prefill(prefixes[:1])
    lg2 = torch.zeros((1, gamma + 1, V), dtype=torch.float32, device=dev)
    gs2.forward(torch.from_numpy(x[:1]).to(dev), gamma, lg2)
    torch.cuda.synchronize()
    so = oracle_model(shape, w)
    st = orc.Stream(so, 160)
    orc.prefill(so, st, prefixes[0])
    assert np.abs(lg2[0].cpu().numpy() - orc.forward(so, st, np.concatenate([[st.pending], x[0]]))).max() < 5e-4


def test_loop_with_an_inherited_draft_emits_what_the_oracle_loop_emits():
    """Algorithm 1 with the paper's kind of draft: the target's lower and upper layers."""
    import dataclasses
    import tests.test_gpu_loop as tl
    from paper_2505_15380_b200 import binding
    shape = synth.ModelShape(6, 128, 4, 2, 64, 256, 300, 8, 1e4)
    layer_map = [0, 5]
    w = synth.make_weights(shape, 23)
    dshape = dataclasses.replace(shape, n_layers=len(layer_map))
    dw = _mapped_weights(w, layer_map)
    tm = binding.Model(shape, synth.weights_blob(shape, w))
    dm = binding.InheritedModel(tm, layer_map)
    otm, odm = oracle_model(shape, w), oracle_model(dshape, dw)
    gamma, n_iter, lens = 3, 12, [30, 66]
    B, V = len(lens), shape.vocab_out
    wl = synth.Workload("inh_loop", shape, dshape, B, gamma, 1.0, 0, tuple(lens), 2, 3, 4)
    cap = max(lens) + n_iter * (gamma + 1) + 16
    ts, ds = binding.Streams(tm, B, cap, gamma), binding.Streams(dm, B, cap, gamma)
    prefixes = [synth.make_prefix(wl, b) for b in range(B)]
    ts.prefill(prefixes)
    ds.prefill(prefixes)
    pool = tl._pool(31, n_iter, B, gamma)
    loop = binding.Loop(ts, ds, prefixes, gamma, pool, 128)
    par = binding.VerifyParams(gamma, 1.0, 0, 0.4)
    ot, od, in_ids = [], [], []
    for b in range(B):
        st, sd = orc.Stream(otm, cap), orc.Stream(odm, cap)
        orc.prefill(otm, st, prefixes[b])
        orc.prefill(odm, sd, prefixes[b])
        sd.length -= 1
        ot.append(st)
        od.append(sd)
        in_ids.append([int(prefixes[b][-2]), int(prefixes[b][-1])])
    matched = 0
    for it in range(n_iter):
        loop.iterate(par)
        torch.cuda.synchronize()
        assert ts.last_status() == 0 and ds.last_status() == 0
        g_x, g_p = loop.draft_tokens.cpu().numpy(), loop.draft_probs.cpu().numpy()
        g_k, g_y = loop.accepted_len.cpu().numpy(), loop.next_token.cpu().numpy()
        for b in range(B):
            ids = np.array(in_ids[b])
            for i in range(gamma):
                lg = orc.forward(odm, od[b], ids)
                od[b].length += len(ids)
                p = orc.transform(lg[-1], 1.0, 0)
                assert np.abs(g_p[b, i] - p).max() < 2e-4       # the draft rows are the inherited model's
                ids = np.array([g_x[b, i]])
            uni = pool[it, b][gamma:].reshape(gamma + 1, 2)
            o = orc.verify(otm, ot[b], g_x[b], g_p[b], uni, temperature=1.0, top_k=0, beta=0.4)
            if all(abs(a - float(uni[i, 0])) >= 1e-3 for i, a in enumerate(o["thresholds"])):
                assert g_k[b] == o["k"]
                matched += 1
            k, y = int(g_k[b]), int(g_y[b])
            orc.commit(ot[b], k, y)
            in_ids[b] = [int(g_x[b, k - 1]) if k > 0 else in_ids[b][1], y]
            od[b].length -= gamma - k
    assert matched >= n_iter * B - 3
