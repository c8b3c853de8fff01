"""The tcgen05 attention of the batched forward (head sizes 64 and 128; forced on, since by
default it serves long key ranges only) at its edges, through the
whole verify step against the float64 oracle: prefixes on both sides of the 64-key tile and of the
page size, a stream with a single cached token, more than 64 query rows per kv head (two row
groups per CTA column), several key splits, contiguous and paged caches.
"""
import pytest

from paper_2505_15380_b200 import synth

pytestmark = pytest.mark.gpu


def _shape(hd, hq, hkv, d=128, f=256, v=300, layers=2):
    return synth.ModelShape(layers, d, hq, hkv, hd, f, v, 8, 1e4, weight_dtype=synth.BF16)


def _wl(shape, batch, gamma, lens, seed):
    return synth.Workload("tc_attention", shape, shape, batch, gamma, 0.8, 25, tuple(lens), 2, seed, seed + 1)


@pytest.mark.parametrize("hd,hq,hkv,gamma,lens", [
    (64, 6, 2, 3, [63, 64, 65, 127, 128, 129, 191, 1]),      # tile and page edges, 32 rows
    (128, 4, 2, 3, [63, 64, 65, 127, 128, 129, 193, 2]),
    (64, 14, 2, 9, [5, 70]),                                 # 7 heads x 10 rows = 70 rows per kv head: two row groups
    (128, 8, 1, 8, [130, 64]),                               # 8 heads x 9 rows = 72 rows, one kv head
    (64, 4, 4, 5, [900, 40, 333]),                           # no grouping (one query head per kv head), long prefix
])
def test_verify_matches_oracle_at_the_edges(hd, hq, hkv, gamma, lens):
    from tests.gpu_case import run_case
    shape = _shape(hd, hq, hkv)
    wl = _wl(shape, len(lens), gamma, lens, seed=hd + hq)
    run_case(wl, beta=0.4, sigma=1.0, commit_and_repeat=True, logit_tol=2e-3, attn_kernel=2)
    pages = sum(-(-(n + gamma + 1) // 64) for n in lens) + len(lens) + 2
    run_case(wl, beta=0.0, sigma=0.5, logit_tol=2e-3, attn_kernel=2,
             paged=(pages, max(-(-(max(lens) + 2 * gamma + 2) // 64) + 1, 4)))


def test_many_key_splits():
    """One stream pair with a long prefix: the grid splits the keys many ways (one wave of CTAs), and
    the last split is ragged."""
    from tests.gpu_case import run_case
    shape = _shape(64, 6, 2)
    wl = _wl(shape, 3, 5, [2500, 1999, 70], seed=5)
    run_case(wl, beta=0.2, sigma=1.0, logit_tol=2e-3, attn_kernel=2)
    run_case(wl, beta=0.2, sigma=1.0, logit_tol=2e-3, attn_kernel=1)   # the warp-level kernel on the same case
