"""cass_draft_gemv_static: the draft GEMV for callers that cannot allocate device memory where they call it (a
plug-in that only receives its tensors, a server whose memory pool is closed after start-up).  Its split-K scratch
is an array built into the library, so the test hands it inputs and outputs only and compares the result with the
ordinary entry point, which takes the scratch from the caller.  Two calls in a row check that what the first call
left in the shared array does not leak into the second.  This file sorts last on purpose."""
import numpy as np
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu


def _encode(cass, w, fmt):
    rows, cols = w.shape
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, rows, cols)
    blob = torch.zeros(bound, dtype=torch.uint8, device="cuda")
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    cass.cass_encode_weights(fmt, w.cuda(), None, blob, ws, status)
    info = cass.cass_weight_blob_info(blob)
    assert int(status.item()) == 0
    return blob, info, status


def test_static_scratch_matches_caller_scratch_twice():
    import paper_2605_26558_b200 as cass
    fmt = cass.default_format()
    cases = [(200, 4096, 11), (70, 688, 12)]          # the second, smaller call runs over the first one's leftovers
    for rows, cols, seed in cases:
        w = synth.student_t_weight(rows, cols, seed, "noalloc/w")
        x = synth.activation_vector(cols, seed, "noalloc/x")[0].cuda()
        blob, info, status = _encode(cass, w, fmt)
        partial = torch.zeros(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device="cuda")
        want32 = torch.zeros(rows, dtype=torch.float32, device="cuda")
        want16 = torch.zeros(rows, dtype=torch.bfloat16, device="cuda")
        cass.cass_draft_gemv(blob, info, x, partial, want16, want32, status)
        got32 = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
        got16 = torch.zeros(rows, dtype=torch.bfloat16, device="cuda")
        cass.cass_draft_gemv_static(blob, info, x, got16, got32, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = want32.cpu().numpy().astype(np.float64)
        rms = float(np.sqrt(np.mean(ref ** 2)))
        err = float(np.abs(got32.cpu().numpy().astype(np.float64) - ref).max())
        assert err <= 1e-4 * rms + 1e-6, (rows, cols, err, rms)
        assert torch.equal(got16, want16)


def test_static_scratch_rejects_oversized_matrices():
    import paper_2605_26558_b200 as cass
    info = cass.BlobInfo()
    info.rows, info.cols, info.n_seg, info.n_rowblocks = 1 << 20, 4096, 2, (1 << 20) // 32
    dummy = torch.zeros(64, dtype=torch.uint8, device="cuda")
    y = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(cass.CassError) as e:
        cass.cass_draft_gemv_static(dummy, info, dummy, None, y, None)
    assert e.value.code == cass.ERR_CAPACITY
