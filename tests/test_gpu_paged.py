"""The paged K/V cache on the GPU (64-token pages from one pool, block tables, O(1) release on
rollback) against the CPU oracle on its plain contiguous cache - the oracle's own paged cache is
pinned bit-identical to that one - plus the page accounting: pages follow the committed lengths,
no page is owned twice, a stream that leaves frees its pages for one that joins."""
import numpy as np
import pytest
import torch

from oracle import ssd_oracle as orc
from paper_2505_15380_b200 import synth
from tests.helpers import oracle_model

pytestmark = pytest.mark.gpu

P = 64


def _shape(hd=64, hq=6, hkv=2, d=128, f=256, v=300, layers=2):
    return synth.ModelShape(layers, d, hq, hkv, hd, f, v, 8, 1e4, weight_dtype=synth.BF16)


def _wl(shape, batch, gamma, lens, temperature=1.0, top_k=0, seed=11):
    return synth.Workload("paged", shape, shape, batch, gamma, temperature, top_k, tuple(lens), 2, seed, seed + 1)


@pytest.mark.parametrize("hd,batch,gamma,lens", [(64, 4, 4, [70, 5, 130, 64]), (128, 2, 3, [1, 200]),
                                                 (32, 6, 5, [63, 64, 65, 127, 128, 129]), (64, 1, 2, [40])])
def test_paged_verify_matches_oracle(hd, batch, gamma, lens):
    """Same parity rules as the contiguous cache: logits, decisions, bit-identical repeats, a commit
    and a second step; forwards of 3 to 36 rows, prefixes on both sides of page boundaries."""
    from tests.gpu_case import run_case
    shape = _shape(hd, hq=4 if hd == 128 else 6)
    wl = _wl(shape, batch, gamma, lens, temperature=0.8, top_k=25)
    run_case(wl, beta=0.4, sigma=1.0, commit_and_repeat=True, paged=(sum(-(-n // P) for n in lens) + batch + 2, 5))
    run_case(wl, beta=0.0, sigma=0.5, paged=(32, 8))


def _check_accounting(gs, n_pages):
    lens, _ = gs.get_state()
    used, free, table = gs.paged_state()
    assert list(used) == [-(-int(n) // P) for n in lens]
    owned = [int(table[b, i]) for b in range(gs.B) for i in range(used[b])]
    assert len(owned) == len(set(owned)) and all(0 <= pg < n_pages for pg in owned)
    assert free == n_pages - len(owned)
    assert (table[np.arange(gs.max_pages)[None, :] >= used[:, None]] == -1).all()
    return used, free


def test_streams_leave_and_join_and_pages_follow_the_lengths():
    from paper_2505_15380_b200 import binding
    shape = _shape()
    w = synth.make_weights(shape, 5)
    om = oracle_model(shape, w)
    gm = binding.Model(shape, synth.weights_blob(shape, w))
    B, gamma, V, n_pages = 3, 4, shape.vocab_out, 9
    gs = binding.PagedStreams(gm, B, n_pages, 4, gamma)
    dev = gm.device
    rng = np.random.default_rng(3)
    prefixes = [rng.integers(0, V, size=n).astype(np.int32) for n in (70, 5, 130)]
    gs.prefill(prefixes)
    ost = []
    for b in range(B):
        st = orc.Stream(om, 4 * P)
        orc.prefill(om, st, prefixes[b])
        ost.append(st)
    _check_accounting(gs, n_pages)
    par = binding.VerifyParams(gamma, 1.0, 0, 0.4)

    def step(seed, compare=(0, 1, 2)):
        p = synth.random_prob_rows(B * gamma, V, seed, sharpness=1.0).reshape(B, gamma, V)
        x = synth.sample_from_rows(p.reshape(-1, V), seed + 1).reshape(B, gamma).astype(np.int32)
        u = synth.verify_uniforms(seed, B, gamma + 1)
        k = torch.zeros(B, dtype=torch.int32, device=dev)
        y = torch.zeros(B, dtype=torch.int32, device=dev)
        lg = torch.zeros((B, gamma + 1, V), dtype=torch.float32, device=dev)
        gs.verify(torch.from_numpy(x).to(dev), torch.from_numpy(p).to(dev), torch.from_numpy(u).to(dev), par, k, y, lg)
        torch.cuda.synchronize()
        assert gs.last_status() == 0
        used, _, _ = gs.paged_state()
        lens, pend = gs.get_state()
        assert list(used) == [-(-(int(n) + gamma + 1) // P) for n in lens]      # provisional rows have pages
        for b in compare:
            ol = orc.forward(om, ost[b], np.concatenate([[ost[b].pending], x[b]]))
            assert np.abs(lg[b].cpu().numpy() - ol).max() < 2e-3
        gs.kv_commit(k, y)
        torch.cuda.synchronize()
        for b in range(B):
            orc.commit(ost[b], int(k[b]), int(y[b]))
        _check_accounting(gs, n_pages)

    for i in range(4):
        step(20 + i)
    # stream 2 rolls back across a page boundary: that page is free at once
    lens, pend = gs.get_state()
    _, free0 = _check_accounting(gs, n_pages)
    assert lens[2] > 2 * P
    new_lens = lens.copy()
    new_lens[2] = P - 3
    gs.kv_truncate(new_lens, pend)
    orc.truncate(ost[2], P - 3, int(pend[2]))
    _, free1 = _check_accounting(gs, n_pages)
    assert free1 == free0 + (-(-int(lens[2]) // P) - 1)
    step(30)
    # stream 0 leaves, a longer prefix joins in its place and reuses the freed pages
    lens, pend = gs.get_state()
    new_lens = lens.copy()
    new_lens[0] = 0
    gs.kv_truncate(new_lens, pend)
    used, free = _check_accounting(gs, n_pages)
    assert used[0] == 0
    joined = rng.integers(0, V, size=150).astype(np.int32)
    gs.prefill_some([joined, None, None])
    ost[0] = orc.Stream(om, 4 * P)
    orc.prefill(om, ost[0], joined)
    _check_accounting(gs, n_pages)
    lens2, pend2 = gs.get_state()
    assert lens2[0] == 149 and pend2[0] == joined[-1] and lens2[1] == lens[1] and lens2[2] == lens[2]
    for i in range(3):
        step(40 + i)            # the other streams' caches survived the churn


def test_exhausted_pool_raises_the_overflow_flag():
    from paper_2505_15380_b200 import binding
    shape = _shape()
    gm = binding.Model(shape, synth.weights_blob(shape, synth.make_weights(shape, 5)))
    gs = binding.PagedStreams(gm, 2, 3, 4, 4)                  # three pages for two streams
    rng = np.random.default_rng(1)
    gs.prefill([rng.integers(0, 300, size=100).astype(np.int32), rng.integers(0, 300, size=120).astype(np.int32)])
    torch.cuda.synchronize()
    assert gs.last_status() & 1                                # 2 + 2 pages wanted, 3 exist
    used, free, _ = gs.paged_state()
    assert free == 0 and used.sum() == 3
