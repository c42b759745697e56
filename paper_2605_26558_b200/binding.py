"""Thin ctypes binding of libcass.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see include/cass.h).  Tensors are torch
CUDA tensors used purely as device buffers; all arithmetic of the method runs inside the library's kernels.
There is no fallback: if the library is missing or cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcass.so")

OK, ERR_INVALID_ARG, ERR_CAPACITY, ERR_UNSUPPORTED, ERR_TIMEOUT, ERR_CUDA = 0, -1, -2, -3, -4, -5
KV_BF16, KV_COMPRESSED = 1, 2
_ERR = {-1: "CASS_ERR_INVALID_ARG", -2: "CASS_ERR_CAPACITY", -3: "CASS_ERR_UNSUPPORTED", -4: "CASS_ERR_TIMEOUT",
        -5: "CASS_ERR_CUDA"}


class CassError(RuntimeError):
    def __init__(self, fn: str, code: int):
        super().__init__(f"{fn} failed: {_ERR.get(code, code)}")
        self.code = code


class Format(C.Structure):
    _fields_ = [("mode", C.c_int), ("w_prune_permille", C.c_int), ("w_trunc_bits", C.c_int),
                ("kv_prune_permille", C.c_int), ("kv_trunc_bits", C.c_int), ("w_seg_cols", C.c_int),
                ("w_chunk_cols", C.c_int), ("kv_mode", C.c_int)]


def default_format(w_p=400, w_t=4, kv_p=400, kv_t=4, seg_cols=0, chunk_cols=0, mode=1, kv_mode=1) -> Format:
    return Format(mode, w_p, w_t, kv_p, kv_t, seg_cols, chunk_cols, kv_mode)


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("hidden", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("ffn", C.c_int), ("vocab", C.c_int), ("max_seq", C.c_int),
                ("max_batch", C.c_int), ("gamma_max", C.c_int), ("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wqkv", "wo", "wgu", "wd", "norm_attn", "norm_ffn")]


class ModelWeights(C.Structure):
    _fields_ = [("h_layers", C.POINTER(LayerWeights)), ("embed", C.c_void_p), ("lm_head", C.c_void_p),
                ("norm_final", C.c_void_p)]


class LayerBlobs(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wqkv", "wo", "wgu", "wd")]


class ModelBlobs(C.Structure):
    _fields_ = [("h_layers", C.POINTER(LayerBlobs)), ("lm_head", C.c_void_p)]


class LayerVdata(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wqkv", "wo", "wgu", "wd")]


class ModelVdata(C.Structure):
    _fields_ = [("h_layers", C.POINTER(LayerVdata)), ("lm_head", C.c_void_p)]


class BlobInfo(C.Structure):
    _fields_ = [("rows", C.c_int), ("cols", C.c_int), ("prune_permille", C.c_int), ("trunc_bits", C.c_int),
                ("seg_cols", C.c_int), ("chunk_cols", C.c_int), ("n_seg", C.c_int), ("n_rowblocks", C.c_int),
                ("kept_per_row", C.c_int), ("max_superblock_bytes", C.c_int), ("mode", C.c_int), ("reserved", C.c_int),
                ("total_bytes", C.c_uint64)]


class BlobStats(C.Structure):
    _fields_ = [("bitmap_bits", C.c_uint64), ("field_bits", C.c_uint64), ("code_bits", C.c_uint64),
                ("total_bits", C.c_uint64)]


class KVView(C.Structure):
    _fields_ = [("fixed", C.c_void_p), ("arena", C.c_void_p), ("offsets", C.c_void_p), ("codebook", C.c_void_p),
                ("k_or_v_bf16", C.c_void_p), ("fixed_words_per_token", C.c_int), ("bitmap_words", C.c_int),
                ("arena_words", C.c_int)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_26558_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    return C.CDLL(LIB_PATH)


lib = _load()
lib.cass_version.restype = C.c_char_p
lib.cass_verify_gemm_scratch_bytes.restype = C.c_size_t
lib.cass_verify_from_parts_scratch_bytes.restype = C.c_size_t
if hasattr(lib, "cass_calib_norms_count"):
    lib.cass_calib_norms_count.restype = C.c_size_t


def _ptr(t) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, int):
        return C.c_void_p(t)
    assert t.is_cuda and t.is_contiguous(), "device buffers must be contiguous CUDA tensors"
    return C.c_void_p(t.data_ptr())


def _stream(stream=None) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(fn: str, rc: int):
    if rc != 0:
        raise CassError(fn, rc)


def cass_version() -> str:
    return lib.cass_version().decode()


def cass_encoded_weight_bytes(fmt: Format, rows: int, cols: int) -> tuple[int, int]:
    bound, ws = C.c_size_t(0), C.c_size_t(0)
    _check("cass_encoded_weight_bytes", lib.cass_encoded_weight_bytes(C.byref(fmt), rows, cols, C.byref(bound), C.byref(ws)))
    return bound.value, ws.value


def cass_encode_weights(fmt: Format, w_bf16, act_norm, blob, workspace, d_status, stream=None):
    rows, cols = w_bf16.shape
    _check("cass_encode_weights", lib.cass_encode_weights(
        C.byref(fmt), _ptr(w_bf16), _ptr(act_norm), rows, cols, _ptr(blob), C.c_size_t(blob.numel() * blob.element_size()),
        _ptr(workspace), C.c_size_t(workspace.numel() * workspace.element_size()), _ptr(d_status), _stream(stream)))


def cass_weight_blob_info(blob, stream=None) -> BlobInfo:
    info = BlobInfo()
    _check("cass_weight_blob_info", lib.cass_weight_blob_info(_ptr(blob), C.byref(info), _stream(stream)))
    return info


def cass_weight_blob_stats(blob, info: BlobInfo, d_scratch, stream=None) -> BlobStats:
    st = BlobStats()
    _check("cass_weight_blob_stats", lib.cass_weight_blob_stats(_ptr(blob), C.byref(info), _ptr(d_scratch), C.byref(st),
                                                                _stream(stream)))
    return st


def cass_decode_weights(blob, info: BlobInfo, out_bf16, stream=None):
    _check("cass_decode_weights", lib.cass_decode_weights(_ptr(blob), C.byref(info), _ptr(out_bf16), _stream(stream)))


def cass_verification_data_bytes(info: BlobInfo) -> int:
    n = C.c_size_t(0)
    _check("cass_verification_data_bytes", lib.cass_verification_data_bytes(C.byref(info), C.byref(n)))
    return n.value


def cass_encode_verification_data(blob, info: BlobInfo, w_bf16, vdata, stream=None):
    _check("cass_encode_verification_data", lib.cass_encode_verification_data(
        _ptr(blob), C.byref(info), _ptr(w_bf16), _ptr(vdata), C.c_size_t(vdata.numel() * vdata.element_size()), _stream(stream)))


def cass_decode_full(blob, info: BlobInfo, vdata, out_bf16, stream=None):
    _check("cass_decode_full", lib.cass_decode_full(_ptr(blob), C.byref(info), _ptr(vdata), _ptr(out_bf16), _stream(stream)))


def cass_draft_gemv(blob, info: BlobInfo, x_bf16, partial, y_bf16, y_f32, d_status, stream=None):
    _check("cass_draft_gemv", lib.cass_draft_gemv(_ptr(blob), C.byref(info), _ptr(x_bf16), _ptr(partial), _ptr(y_bf16),
                                                  _ptr(y_f32), _ptr(d_status), _stream(stream)))


def cass_draft_gemv_batch(blob, info: BlobInfo, x_bf16, n_vec: int, partial, y_bf16, y_f32, d_status, stream=None):
    _check("cass_draft_gemv_batch", lib.cass_draft_gemv_batch(_ptr(blob), C.byref(info), _ptr(x_bf16), n_vec, _ptr(partial),
                                                              _ptr(y_bf16), _ptr(y_f32), _ptr(d_status), _stream(stream)))


def cass_draft_gemv_static(blob, info: BlobInfo, x_bf16, y_bf16, y_f32, d_status, stream=None):
    """cass_draft_gemv with the partial sums in the library's built-in scratch: nothing is allocated, here or there."""
    _check("cass_draft_gemv_static", lib.cass_draft_gemv_static(_ptr(blob), C.byref(info), _ptr(x_bf16), _ptr(y_bf16),
                                                                _ptr(y_f32), _ptr(d_status), _stream(stream)))


def cass_session_bytes(desc: ModelDesc, fmt: Format) -> int:
    n = C.c_size_t(0)
    _check("cass_session_bytes", lib.cass_session_bytes(C.byref(desc), C.byref(fmt), C.byref(n)))
    return n.value


def cass_session_init(mem, desc: ModelDesc, fmt: Format, weights: ModelWeights, blobs, stream=None) -> C.c_void_p:
    h = C.c_void_p(0)
    _check("cass_session_init", lib.cass_session_init(
        _ptr(mem), C.c_size_t(mem.numel() * mem.element_size()), C.byref(desc), C.byref(fmt), C.byref(weights),
        C.byref(blobs) if blobs is not None else None, C.byref(h), _stream(stream)))
    return h


def cass_session_set_blobs(session, blobs: ModelBlobs, stream=None):
    _check("cass_session_set_blobs", lib.cass_session_set_blobs(session, C.byref(blobs), _stream(stream)))


def cass_verify_from_parts_scratch_bytes(desc: ModelDesc) -> int:
    return int(lib.cass_verify_from_parts_scratch_bytes(C.byref(desc)))


def cass_session_verify_from_parts(session, vdata, scratch_bf16):
    if vdata is None:
        _check("cass_session_verify_from_parts", lib.cass_session_verify_from_parts(session, None, None, C.c_size_t(0)))
        return
    _check("cass_session_verify_from_parts", lib.cass_session_verify_from_parts(
        session, C.byref(vdata), _ptr(scratch_bf16), C.c_size_t(scratch_bf16.numel() * scratch_bf16.element_size())))


def cass_session_destroy(session):
    _check("cass_session_destroy", lib.cass_session_destroy(session))


def cass_session_reset(session, stream=None):
    _check("cass_session_reset", lib.cass_session_reset(session, _stream(stream)))


def cass_session_status(session, stream=None) -> tuple[int, int]:
    st, ln = C.c_int32(0), C.c_int32(0)
    _check("cass_session_status", lib.cass_session_status(session, C.byref(st), C.byref(ln), _stream(stream)))
    return st.value, ln.value


def cass_session_lens(session, batch: int, stream=None) -> list[int]:
    buf = (C.c_int32 * max(batch, 8))()
    _check("cass_session_lens", lib.cass_session_lens(session, buf, _stream(stream)))
    return [int(buf[i]) for i in range(batch)]


def cass_session_rows(desc: ModelDesc) -> int:
    r = int(lib.cass_session_rows(C.byref(desc)))
    if r < 0:
        raise CassError("cass_session_rows", r)
    return r


def cass_calib_enable(session, on: bool, stream=None):
    _check("cass_calib_enable", lib.cass_calib_enable(session, int(on), _stream(stream)))


def cass_calib_norms_count(desc: ModelDesc) -> int:
    return int(lib.cass_calib_norms_count(C.byref(desc)))


def cass_calib_norms(session, norms_out, stream=None):
    _check("cass_calib_norms", lib.cass_calib_norms(session, _ptr(norms_out), _stream(stream)))


def cass_kv_append(session, layer: int, k_bf16, v_bf16, start_pos: int, n_new: int, flags: int, stream=None, seq: int = 0):
    _check("cass_kv_append", lib.cass_kv_append(session, seq, layer, _ptr(k_bf16), _ptr(v_bf16), start_pos, n_new, flags,
                                                _stream(stream)))


def cass_kv_build_codebook(session, n_tokens: int, stream=None):
    _check("cass_kv_build_codebook", lib.cass_kv_build_codebook(session, n_tokens, _stream(stream)))


def cass_set_len(session, n: int, stream=None):
    _check("cass_set_len", lib.cass_set_len(session, n, _stream(stream)))


def cass_set_lens(session, lens, stream=None):
    buf = (C.c_int32 * 8)(*[int(v) for v in lens])
    _check("cass_set_lens", lib.cass_set_lens(session, buf, _stream(stream)))


def cass_draft_step(session, tok_in, tok_out, logits_opt=None, stream=None, tok_stride: int = 1):
    _check("cass_draft_step", lib.cass_draft_step(session, _ptr(tok_in), _ptr(tok_out), tok_stride, _ptr(logits_opt),
                                                  _stream(stream)))


def cass_verify(session, toks, g: int, target_argmax, logits_opt=None, stream=None):
    _check("cass_verify", lib.cass_verify(session, _ptr(toks), g, _ptr(target_argmax), _ptr(logits_opt), _stream(stream)))


def cass_draft_attention(session, layer: int, q_bf16, out_bf16, stream=None):
    _check("cass_draft_attention", lib.cass_draft_attention(session, layer, _ptr(q_bf16), _ptr(out_bf16), _stream(stream)))


def cass_verify_gemm_scratch_bytes(n: int, k: int) -> int:
    return int(lib.cass_verify_gemm_scratch_bytes(n, k))


def cass_verify_gemm(w_bf16, x_bf16, rows: int, scratch, y_bf16, y_f32, d_status, stream=None):
    n, k = w_bf16.shape
    assert x_bf16.shape[0] == (16 if rows <= 16 else 32 if rows <= 32 else 64) and x_bf16.shape[1] == k
    _check("cass_verify_gemm", lib.cass_verify_gemm(_ptr(w_bf16), _ptr(x_bf16), rows, n, k, _ptr(scratch),
                                                    C.c_size_t(scratch.numel() * scratch.element_size()), _ptr(y_bf16),
                                                    _ptr(y_f32), _ptr(d_status), _stream(stream)))


def cass_accept(session, draft, target_argmax, g: int, n_accepted, out_tokens, next_tok, stream=None,
                draft_stride: int | None = None, next_stride: int = 1):
    _check("cass_accept", lib.cass_accept(session, _ptr(draft), g if draft_stride is None else draft_stride,
                                          _ptr(target_argmax), g, _ptr(n_accepted), _ptr(out_tokens), _ptr(next_tok),
                                          next_stride, _stream(stream)))


def cass_accept_sampling(session, n_seq: int, draft, p_target, q_draft, vocab: int, r_uniform, u_uniform, g: int,
                         n_accepted, out_tokens, next_tok, stream=None, draft_stride: int | None = None,
                         next_stride: int = 1):
    _check("cass_accept_sampling", lib.cass_accept_sampling(
        session, n_seq, _ptr(draft), g if draft_stride is None else draft_stride, _ptr(p_target), _ptr(q_draft), vocab,
        _ptr(r_uniform), _ptr(u_uniform), g, _ptr(n_accepted), _ptr(out_tokens), _ptr(next_tok), next_stride,
        _stream(stream)))


def cass_softmax(logits, rows: int, vocab: int, temperature: float, probs, stream=None):
    _check("cass_softmax", lib.cass_softmax(_ptr(logits), rows, vocab, C.c_float(temperature), _ptr(probs), _stream(stream)))


def cass_sample(probs, rows: int, vocab: int, u, tokens, stream=None, tok_stride: int = 1):
    _check("cass_sample", lib.cass_sample(_ptr(probs), rows, vocab, _ptr(u), _ptr(tokens), tok_stride, _stream(stream)))


def cass_kv_query(session, layer: int, kind: int, head: int, seq: int = 0) -> KVView:
    v = KVView()
    _check("cass_kv_query", lib.cass_kv_query(session, seq, layer, kind, head, C.byref(v)))
    return v


def cass_debug_activation(session, which: int) -> tuple[int, int, int]:
    p, r, c = C.c_void_p(0), C.c_int(0), C.c_int(0)
    _check("cass_debug_activation", lib.cass_debug_activation(session, which, C.byref(p), C.byref(r), C.byref(c)))
    return p.value, r.value, c.value
