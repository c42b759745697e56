"""GPU parity: weight encoder (bit-exact blob), decode hook, draft GEMV -- against the CPU oracle."""
import numpy as np
import pytest
import torch

import synth
from oracle import codec, layout

pytestmark = pytest.mark.gpu


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().astype(np.uint16)


@pytest.fixture(scope="module")
def cass():
    import paper_2605_26558_b200 as m
    assert torch.cuda.is_available()
    return m


def _encode_gpu(cass, w: torch.Tensor, act, fmt):
    dev = "cuda"
    rows, cols = w.shape
    bound, ws_bytes = cass.cass_encoded_weight_bytes(fmt, rows, cols)
    blob = torch.zeros(bound // 4 + 64, dtype=torch.int32, device=dev)
    ws = torch.zeros(ws_bytes // 4 + 64, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    wd = w.to(dev)
    ad = None if act is None else torch.from_numpy(act).to(dev)
    cass.cass_encode_weights(fmt, wd, ad, blob, ws, status)
    info = cass.cass_weight_blob_info(blob)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return blob, info, status


CASES = [
    # rows, cols, p, t, seg, chunk
    (70, 688, 400, 4, 512, 128),          # ragged rows and columns, several segments
    (96, 1024, 400, 4, 0, 0),
    (64, 256, 400, 4, 0, 0),
    (33, 704, 0, 0, 0, 0),                # identity format
    (40, 512, 300, 5, 256, 64),           # 3-bit fields: ten per word, packed (not rotated)
    (96, 2048, 400, 1, 0, 0),             # 7-bit fields: four per word, chunks that start inside a field word
    (70, 1376, 500, 2, 1024, 128),        # 6-bit fields: five per word
    (64, 4096, 300, 3, 0, 0),             # 5-bit fields: six per word, two full segments
    (32, 4096, 600, 5, 2048, 64),         # 3-bit fields, 60 % pruned: long gaps between kept columns
    (128, 4096, 400, 4, 0, 0),            # Llama-3-8B hidden size: two full segments
    (64, 4096, 500, 0, 1024, 256),
]


@pytest.mark.parametrize("rows,cols,p,t,seg,chunk", CASES)
def test_encode_decode_gemv(cass, rows, cols, p, t, seg, chunk):
    w = synth.student_t_weight(rows, cols, 0, f"gpu/w{rows}x{cols}")
    rng = np.random.default_rng(rows * 7 + cols)
    act = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    wb = _bits(w)
    fmt = cass.default_format(w_p=p, w_t=t, seg_cols=seg, chunk_cols=chunk)
    blob, info, status = _encode_gpu(cass, w, act, fmt)
    want, oinfo = layout.encode_weight_blob(wb, act, p, t, seg_cols=seg or 2048, chunk_cols=chunk or 256)
    got = blob[: info.total_bytes // 4].cpu().numpy().view(np.uint32)
    assert info.total_bytes == want.size * 4
    assert (info.rows, info.cols, info.seg_cols, info.chunk_cols) == (rows, cols, oinfo["seg_cols"], oinfo["chunk_cols"])
    assert np.array_equal(got[:32], want[:32]), "header"
    assert np.array_equal(got[32:96], want[32:96]), "codebook"
    assert np.array_equal(got, want), "blob bytes"

    # decode hook == zero-padded reconstruction of the speculation data
    out = torch.empty(rows, cols, dtype=torch.bfloat16, device="cuda")
    cass.cass_decode_weights(blob, info, out)
    dec = _bits(out)
    assert np.array_equal(dec, codec.draft_bits(wb, oinfo["keep"], t))

    # draft GEMV against the oracle's fp64 product on the decoded matrix
    x = synth.activation_vector(cols, 1, "gpu/x")[0]
    xd = x.cuda()
    n_pad = info.n_rowblocks * 32
    partial = torch.zeros(info.n_seg * n_pad, dtype=torch.float32, device="cuda")
    y32 = torch.zeros(rows, dtype=torch.float32, device="cuda")
    y16 = torch.zeros(rows, dtype=torch.bfloat16, device="cuda")
    cass.cass_draft_gemv(blob, info, xd, partial, y16, y32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = codec.bf16_bits_to_f64(dec) @ codec.bf16_bits_to_f64(_bits(x))
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(y32.cpu().numpy().astype(np.float64) - ref).max()
    assert err <= 2e-2 * rms, (err, rms)
    assert err <= 1e-4 * rms + 1e-6, (err, rms)          # fp32 accumulation is far tighter than the bar
    assert np.array_equal(_bits(y16), codec.f64_to_bf16_bits(y32.cpu().numpy().astype(np.float64)))


def test_long_gaps_and_long_codewords(cass):
    """Rows with long zero runs in the bitmap and very rare exponents (long codewords): the window walk of the
    draft GEMV has to fall back to its careful walk for those groups."""
    rows, cols = 64, 1024
    w = synth.student_t_weight(rows, cols, 3, "gpu/irregular").float()
    w[3, 100:400] = 0.0                       # pruned run longer than a 32-bit window
    w[5, :] *= 1e-3
    w[7, ::5] *= 2.0 ** 40                    # exponents that are rare in the matrix: long codes
    w[9, 17] = 3.0e38
    w[11, :] = 0.0                            # all-zero row: every score ties
    w = w.to(torch.bfloat16)
    wb = _bits(w)
    fmt = cass.default_format()
    blob, info, status = _encode_gpu(cass, w, None, fmt)
    want, oinfo = layout.encode_weight_blob(wb, None, 400, 4)
    got = blob[: info.total_bytes // 4].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want)
    inv = codec.invert_codebook(oinfo["codebook"])
    code_len = inv[(wb >> 7) & 0xFF] + 1
    assert (code_len[7][oinfo["keep"][7]] > 8).any() and not oinfo["keep"][3, 100:400].any(), "the case should be hard"
    x = synth.activation_vector(cols, 2, "gpu/x2")[0]
    partial = torch.zeros(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device="cuda")
    y32 = torch.zeros(rows, dtype=torch.float32, device="cuda")
    cass.cass_draft_gemv(blob, info, x.cuda(), partial, None, y32, status)
    torch.cuda.synchronize()
    dec = layout.decode_weight_blob(want)
    ref = codec.bf16_bits_to_f64(dec) @ codec.bf16_bits_to_f64(_bits(x))
    got_y = y32.cpu().numpy().astype(np.float64)
    scale = np.abs(codec.bf16_bits_to_f64(dec)) @ np.abs(codec.bf16_bits_to_f64(_bits(x)))
    assert (np.abs(got_y - ref) <= 1e-5 * scale + 1e-30).all()


def test_full_size_down_projection(cass):
    """Llama-3-8B down projection (4096 x 14336: seven column segments, the launch configuration the benchmark
    times): sampled superblocks bit-exact against the oracle, every GEMV output against the oracle's fp64 product."""
    rows, cols = 4096, 14336
    w = synth.student_t_weight(rows, cols, 21, "gpu/full_wd")
    rng = np.random.default_rng(5)
    act = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    wb = _bits(w)
    fmt = cass.default_format()
    blob, info, status = _encode_gpu(cass, w, act, fmt)
    sample = [0, 1, 63, 127]
    bodies, oinfo = layout.encode_weight_blob(wb, act, 400, 4, rowblocks=sample)
    got = blob[: info.total_bytes].cpu().numpy().view(np.uint32)
    assert np.array_equal(got[32:96].view(np.uint8), oinfo["codebook"])
    n_sb = info.n_rowblocks * info.n_seg
    directory = got[96: 96 + 4 * n_sb].reshape(n_sb, 4)
    for sb, (body, w_f, w_u, w3) in bodies.items():
        off = int(directory[sb][0]) * 4
        assert tuple(int(x) for x in directory[sb][1:]) == (w_f, w_u, w3), sb
        assert np.array_equal(got[off: off + body.size], body), sb
    x = synth.activation_vector(cols, 3, "gpu/full_x")[0]
    partial = torch.zeros(info.n_seg * info.n_rowblocks * 32, dtype=torch.float32, device="cuda")
    y32 = torch.zeros(rows, dtype=torch.float32, device="cuda")
    cass.cass_draft_gemv(blob, info, x.cuda(), partial, None, y32, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    dec = codec.draft_bits(wb, oinfo["keep"], 4)
    ref = codec.bf16_bits_to_f64(dec) @ codec.bf16_bits_to_f64(_bits(x))
    rms = float(np.sqrt(np.mean(ref ** 2)))
    err = np.abs(y32.cpu().numpy().astype(np.float64) - ref).max()
    assert err <= 2e-2 * rms and err <= 1e-4 * rms + 1e-6, (err, rms)


@pytest.mark.parametrize("rows,cols,p,t,seg,chunk", [(70, 688, 400, 4, 512, 128), (33, 1000, 300, 5, 256, 64),
                                                      (40, 704, 0, 0, 0, 0), (64, 4096, 400, 4, 0, 0)])
def test_verification_data_and_exact_reconstruction(cass, rows, cols, p, t, seg, chunk):
    """Verification data (low mantissa bits of kept values, raw pruned values) bit-exact against the oracle's, and
    speculation data + verification data decoded back to the original bf16 matrix bit for bit (Sec. 4.1)."""
    w = synth.student_t_weight(rows, cols, 4, f"gpu/vd{rows}x{cols}")
    rng = np.random.default_rng(rows + cols)
    act = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    wb = _bits(w)
    fmt = cass.default_format(w_p=p, w_t=t, seg_cols=seg, chunk_cols=chunk)
    blob, info, _ = _encode_gpu(cass, w, act, fmt)
    nbytes = cass.cass_verification_data_bytes(info)
    keep = codec.keep_mask_weights(wb, act, p)
    want = layout.encode_verification_data(wb, keep, p, t)
    assert nbytes == want.size * 4
    vdata = torch.full((nbytes // 4,), -1, dtype=torch.int32, device="cuda")
    cass.cass_encode_verification_data(blob, info, w.cuda(), vdata)
    assert np.array_equal(vdata.cpu().numpy().view(np.uint32), want)
    full = torch.zeros(rows, cols, dtype=torch.bfloat16, device="cuda")
    cass.cass_decode_full(blob, info, vdata, full)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(full), wb)
    # both parts together hold fewer bits than the bf16 matrix (the memory claim of Sec. 7.2): the exponent code saves
    # more than the bitmap costs
    st = cass.cass_weight_blob_stats(blob, info, torch.zeros(8, dtype=torch.uint8, device="cuda"))
    kept = info.kept_per_row
    content = st.bitmap_bits + st.field_bits + st.code_bits + rows * (kept * t + (cols - kept) * 16)
    assert content < 16 * rows * cols
