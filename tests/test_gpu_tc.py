"""The tcgen05 projection kernel of the batched forward, alone, against float64 matrix products.

The kernel computes acc[t, r] = sum_k x[t, k] * w[r, k] with bf16 weights and fp32 activations that
enter the tensor cores as a bf16 leading part plus a bf16 remainder; the reference is the plain
definition in float64 (numpy matmul).  Shapes cover one and several 128-row tiles with a ragged
last tile, K that is not a multiple of the 16-column k-step, K splits, token counts on both sides
of the 256-column limit of one instruction, and the three epilogues.
"""
import numpy as np
import pytest
import torch

from paper_2505_15380_b200 import synth

pytestmark = pytest.mark.gpu


def _data(M, n_rows, K, seed):
    rng = np.random.Generator(np.random.Philox(key=seed))
    w = synth.bf16_round((rng.standard_normal((n_rows, K)) * 0.05).astype(np.float32))
    x = rng.standard_normal((M, K)).astype(np.float32)
    dev = torch.device("cuda:0")
    return w, x, torch.from_numpy(w).to(dev).to(torch.bfloat16), torch.from_numpy(x).to(dev)


def _tol(ref):
    # two-term bf16 split of x: each product is exact to ~2^-17 relative; fp32 accumulation
    return 3e-5 * float(np.abs(ref).max()) + 1e-6


@pytest.mark.parametrize("M,n_rows,K,ksplit", [
    (96, 1152, 896, 3), (17, 130, 200, 1), (448, 256, 512, 4), (272, 128, 64, 2), (512, 384, 256, 1),
    (33, 896, 4864, 21), (1, 128, 16, 1), (240, 640, 1536, 6)])
def test_partial_sums_add_up_to_the_product(M, n_rows, K, ksplit):
    from paper_2505_15380_b200 import binding
    w, x, dw, dx = _data(M, n_rows, K, seed=M + n_rows)
    out, status = binding.tc_gemm_check(dw, dx, ksplit, 0)
    out2, _ = binding.tc_gemm_check(dw, dx, ksplit, 0)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    assert torch.equal(out, out2)                                  # bit-reproducible
    acc = out.double().sum(dim=0).cpu().numpy()[:M, :n_rows]
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(acc - ref).max() <= _tol(ref)
    if ksplit > 1:                                                 # the slices really are partial
        assert np.abs(out[0].double().cpu().numpy()[:M, :n_rows] - ref).max() > 10 * _tol(ref)


@pytest.mark.parametrize("M,n_rows,K", [(96, 6564, 896), (20, 300, 64), (300, 515, 128)])
def test_store_epilogue_gives_logit_layout(M, n_rows, K):
    from paper_2505_15380_b200 import binding
    w, x, dw, dx = _data(M, n_rows, K, seed=7)
    out, status = binding.tc_gemm_check(dw, dx, 1, 1)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    ref = x.astype(np.float64) @ w.astype(np.float64).T
    assert np.abs(out.double().cpu().numpy() - ref).max() <= _tol(ref)


@pytest.mark.parametrize("M,F,K", [(96, 304, 128), (18, 100, 64), (448, 136, 256)])
def test_swiglu_epilogue_writes_a_packed_operand(M, F, K):
    """Weight rows (gate_j, up_j) interleaved; the output is SiLU(gate) * up as the next projection's
    operand: bf16 leading part and remainder in the layout include/ssd.h states."""
    from paper_2505_15380_b200 import binding
    w, x, dw, dx = _data(M, 2 * F, K, seed=11)
    out, status = binding.tc_gemm_check(dw, dx, 1, 2)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    acc = x.astype(np.float64) @ w.astype(np.float64).T
    gate, up = acc[:, 0::2], acc[:, 1::2]
    ref = gate / (1.0 + np.exp(-gate)) * up
    raw = out.cpu().numpy().view(np.uint16)                        # bf16 bit patterns
    Mpad = (M + 15) // 16 * 16
    chunks = 1 if Mpad <= 256 else (Mpad + 255) // 256       # rows are stored in chunks of Mc
    Mc = Mpad if chunks == 1 else ((Mpad + chunks - 1) // chunks + 15) // 16 * 16
    KS = (F + 15) // 16
    t = np.arange(M)[:, None]
    j = np.arange(F)[None, :]
    base = ((t // Mc) * KS + j // 16) * (Mc * 64) + ((j // 8) % 2) * (Mc * 32) + (t % Mc) * 16 + (j % 8) * 2
    hi = synth.from_bf16_bits(raw[(base // 2)]).astype(np.float64)
    lo = synth.from_bf16_bits(raw[((base + Mc * 16) // 2)]).astype(np.float64)
    assert np.abs(hi + lo - ref).max() <= 3e-5 * np.abs(ref).max() + 1e-6
    assert np.abs(hi - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-6     # hi alone is the bf16 rounding
    assert np.abs(lo).max() > 0


def test_bad_sizes_are_refused():
    from paper_2505_15380_b200 import binding
    L = binding.lib()
    assert L.ssd_tc_gemm_scratch_bytes(513, 128, 64) == 0
    assert L.ssd_tc_gemm_scratch_bytes(16, 128, 60) == 0
    dev = torch.device("cuda:0")
    w = torch.zeros((128, 64), dtype=torch.bfloat16, device=dev)
    x = torch.zeros((16, 64), dtype=torch.float32, device=dev)
    with pytest.raises(binding.SsdError, match="parameter"):
        binding.tc_gemm_check(w, x, 5, 0)          # more K slices than k-steps
    with pytest.raises(binding.SsdError, match="parameter"):
        binding.tc_gemm_check(w, x, 2, 1)          # a K split needs the partial-sum epilogue
