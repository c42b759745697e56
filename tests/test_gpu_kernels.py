"""Kernel-level GPU parity on identical inputs: verification GEMM (tcgen05) against the oracle's fp64 product."""
import numpy as np
import pytest
import torch

import synth
from oracle import codec

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().astype(np.uint16)


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    return m


def _run(cass, w, x16, rows):
    n, k = w.shape
    scratch = torch.empty(cass.cass_verify_gemm_scratch_bytes(n, k), dtype=torch.uint8, device="cuda")
    y32 = torch.full((rows, n), float("nan"), dtype=torch.float32, device="cuda")
    y16 = torch.zeros(rows, n, dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_verify_gemm(w, x16, rows, scratch, y16, y32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return y32, y16


@pytest.mark.parametrize("n,k,rows", [(1024, 256, 1), (1376, 688, 5), (1000, 264, 16), (4096, 4096, 5),
                                      (384, 14336, 3), (6144, 4096, 9)])
def test_verify_gemm_against_oracle(cass, n, k, rows):
    w = synth.student_t_weight(n, k, 5, f"vg/w{n}x{k}")
    x = synth.activation_vector(k, 6, f"vg/x{k}", rows=16)
    y32, y16 = _run(cass, w.cuda(), x.cuda().contiguous(), rows)
    ref = codec.bf16_bits_to_f64(_bits(x[:rows])) @ codec.bf16_bits_to_f64(_bits(w)).T
    got = y32.cpu().numpy().astype(np.float64)
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = float(np.abs(got - ref).max())
    assert err <= TOL * rms, (err, rms)
    assert err <= 1e-4 * rms + 1e-6, (err, rms)              # fp32 accumulation is far inside the bar
    assert np.array_equal(_bits(y16), codec.f64_to_bf16_bits(got))


def test_verify_gemm_rows_do_not_depend_on_the_batch(cass):
    n, k = 2048, 1024
    w = synth.student_t_weight(n, k, 7, "vg/inv").cuda()
    x = synth.activation_vector(k, 8, "vg/invx", rows=16).cuda().contiguous()
    full, _ = _run(cass, w, x, 16)
    for rows in (1, 5, 9):
        part, _ = _run(cass, w, x, rows)
        assert torch.equal(part, full[:rows])
    x2 = x.clone()
    x2[1:] = float("nan")                                      # other rows' contents cannot leak into row 0
    alone, _ = _run(cass, w, x2, 1)
    assert torch.equal(alone[0], full[0])
