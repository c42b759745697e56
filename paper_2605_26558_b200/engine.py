"""Step sequencing on top of the C boundary: what a user of the library writes.

This module only allocates device buffers (torch) and calls the entry points of libcass.so in order; every
arithmetic step (encoding, draft pass, verification, acceptance) runs in the library's kernels.
"""
from __future__ import annotations

import ctypes as C
import dataclasses

import torch

from . import binding as B


@dataclasses.dataclass
class StepStats:
    steps: int = 0
    accepted: int = 0
    emitted: int = 0

    @property
    def mean_accepted(self) -> float:
        return self.accepted / max(self.steps, 1)


def fuse_layer_weights(lw: dict) -> dict:
    """q, k, v rows stacked into one matrix, gate and up rows stacked into one matrix (layout only)."""
    return {
        "wqkv": torch.cat([lw["wq"], lw["wk"], lw["wv"]], dim=0).contiguous(),
        "wo": lw["wo"].contiguous(),
        "wgu": torch.cat([lw["wg"], lw["wu"]], dim=0).contiguous(),
        "wd": lw["wd"].contiguous(),
        "norm_attn": lw["norm_attn"].contiguous(),
        "norm_ffn": lw["norm_ffn"].contiguous(),
    }


class Engine:
    """`batch` sequences (1, 2, 4 or 8) decoded together on one GPU.  `weights` = {"layers": [fused layer dicts],
    "embed", "lm_head", "norm_final"} of bf16 CUDA tensors (see fuse_layer_weights).  With batch = 1 the token-level
    results (prefill's return, generate's list) are plain ints; with more they are per-sequence lists."""

    def __init__(self, shape, weights: dict, fmt: B.Format | None = None, max_seq: int = 1024, gamma_max: int = 8,
                 device="cuda", batch: int = 1):
        self.shape, self.w, self.device = shape, weights, torch.device(device)
        self.fmt = fmt if fmt is not None else B.default_format()
        self.batch = batch
        self.desc = B.ModelDesc(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                shape.ffn, shape.vocab, max_seq, batch, gamma_max, shape.rope_theta, shape.rms_eps)
        self.max_rows = B.cass_session_rows(self.desc)
        nbytes = B.cass_session_bytes(self.desc, self.fmt)
        self.mem = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self._lw = (B.LayerWeights * shape.n_layers)()
        for i, lw in enumerate(weights["layers"]):
            for name in ("wqkv", "wo", "wgu", "wd", "norm_attn", "norm_ffn"):
                assert lw[name].dtype == torch.bfloat16 and lw[name].is_cuda and lw[name].is_contiguous()
                setattr(self._lw[i], name, lw[name].data_ptr())
        self._mw = B.ModelWeights(self._lw, weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                                  weights["norm_final"].data_ptr())
        self.session = B.cass_session_init(self.mem, self.desc, self.fmt, self._mw, None)
        self.blobs = None
        self.n_prompt = 0
        # step buffers, [batch][gamma + 1] for the gamma in use: toks[b][0] = last emitted token of sequence b,
        # toks[b][1..g] = its drafted tokens
        self.toks = torch.zeros(64, dtype=torch.int32, device=self.device)
        self.targ = torch.zeros(64, dtype=torch.int32, device=self.device)
        self.out_tokens = torch.zeros(64, dtype=torch.int32, device=self.device)
        self.n_acc = torch.zeros(8, dtype=torch.int32, device=self.device)
        self._stride = 1              # gamma + 1 of the layout the token buffers are in
        self._graphs = {}

    def close(self):
        if self.session is not None:
            B.cass_session_destroy(self.session)
            self.session = None

    # ------------------------------------------------------------------ set-up
    def reset(self):
        B.cass_session_reset(self.session)
        self.n_prompt = 0

    def prefill(self, prompt: torch.Tensor, calibrate: bool = False):
        """Target pass over the prompt(s) ([n] or [batch][n] token ids, equal lengths) in chunks of up to 16 rows per
        sequence (bf16 cache only); returns the first generated token (per sequence).  With calibrate, the Wanda
        activation statistics are accumulated on the way."""
        prompt = prompt.to(self.device, torch.int32).reshape(self.batch, -1).contiguous()
        n = int(prompt.shape[1])
        chunk = min(16, self.max_rows // self.batch)
        B.cass_calib_enable(self.session, calibrate)
        pos, rows = 0, 0
        while pos < n:
            rows = min(chunk, n - pos)
            B.cass_set_len(self.session, pos)
            B.cass_verify(self.session, prompt[:, pos: pos + rows].contiguous(), rows - 1, self.targ)
            pos += rows
        B.cass_calib_enable(self.session, False)
        B.cass_set_len(self.session, n)
        self.n_prompt = n
        first = self.targ[: self.batch * rows].view(self.batch, rows)[:, rows - 1].clone()
        self._stride = 1
        self.toks[: self.batch] = first
        return int(first[0].item()) if self.batch == 1 else first.tolist()

    def calib_norms(self) -> dict:
        cnt = B.cass_calib_norms_count(self.desc)
        buf = torch.empty(cnt, dtype=torch.float32, device=self.device)
        B.cass_calib_norms(self.session, buf)
        s = self.shape
        kmax = max(s.hidden, s.ffn, s.n_q_heads * s.head_dim)
        per_layer = buf[: s.n_layers * 4 * kmax].view(s.n_layers, 4, kmax)
        cols = (s.hidden, s.n_q_heads * s.head_dim, s.hidden, s.ffn)
        names = ("wqkv", "wo", "wgu", "wd")
        return {"layers": [{nm: per_layer[l, i, :cols[i]].contiguous() for i, nm in enumerate(names)}
                           for l in range(s.n_layers)],
                "lm_head": buf[s.n_layers * 4 * kmax:].contiguous()}

    def encode_weights(self, norms: dict | None):
        """Runs the GPU weight encoder on the four matrices of every layer and on lm_head."""
        status = torch.zeros(1, dtype=torch.int32, device=self.device)
        blobs = {"layers": [], "infos": {}}
        ws = None

        def enc(w, a):
            nonlocal ws
            bound, ws_bytes = B.cass_encoded_weight_bytes(self.fmt, w.shape[0], w.shape[1])
            if ws is None or ws.numel() < ws_bytes:
                ws = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
            blob = torch.empty(bound, dtype=torch.uint8, device=self.device)
            B.cass_encode_weights(self.fmt, w, a, blob, ws, status)
            info = B.cass_weight_blob_info(blob)
            return blob[: info.total_bytes].clone(), info

        for l, lw in enumerate(self.w["layers"]):
            d = {}
            for nm in ("wqkv", "wo", "wgu", "wd"):
                a = None if norms is None or norms["layers"][l].get(nm) is None else \
                    norms["layers"][l][nm].to(self.device, torch.float32).contiguous()
                d[nm], blobs["infos"][(l, nm)] = enc(lw[nm], a)
            blobs["layers"].append(d)
        a = None if norms is None or norms.get("lm_head") is None else \
            norms["lm_head"].to(self.device, torch.float32).contiguous()
        blobs["lm_head"], blobs["infos"]["lm_head"] = enc(self.w["lm_head"], a)
        if int(status.item()) != 0:
            raise B.CassError("cass_encode_weights(status)", int(status.item()))
        self.set_blobs(blobs)
        return blobs

    def set_blobs(self, blobs: dict):
        self.blobs = blobs
        self._lb = (B.LayerBlobs * self.shape.n_layers)()
        for i, d in enumerate(blobs["layers"]):
            for nm in ("wqkv", "wo", "wgu", "wd"):
                setattr(self._lb[i], nm, d[nm].data_ptr())
        self._mb = B.ModelBlobs(self._lb, blobs["lm_head"].data_ptr())
        B.cass_session_set_blobs(self.session, self._mb)

    def verify_from_parts(self, drop_bf16: bool = False) -> int:
        """Encodes the verification data of every matrix and makes the session verify from speculation + verification
        data instead of the bf16 copy (needs encode_weights first).  With drop_bf16 the engine lets go of the bf16
        projection matrices (embeddings and norm gains stay).  Returns the bytes of verification data."""
        assert self.blobs is not None
        self.vdata = {"layers": []}
        total = 0

        def enc(blob, info, w):
            nonlocal total
            buf = torch.empty(B.cass_verification_data_bytes(info), dtype=torch.uint8, device=self.device)
            B.cass_encode_verification_data(blob, info, w, buf)
            total += buf.numel()
            return buf

        for l, lw in enumerate(self.w["layers"]):
            self.vdata["layers"].append({nm: enc(self.blobs["layers"][l][nm], self.blobs["infos"][(l, nm)], lw[nm])
                                         for nm in ("wqkv", "wo", "wgu", "wd")})
        self.vdata["lm_head"] = enc(self.blobs["lm_head"], self.blobs["infos"]["lm_head"], self.w["lm_head"])
        self._lv = (B.LayerVdata * self.shape.n_layers)()
        for i, d in enumerate(self.vdata["layers"]):
            for nm in ("wqkv", "wo", "wgu", "wd"):
                setattr(self._lv[i], nm, d[nm].data_ptr())
        self._mv = B.ModelVdata(self._lv, self.vdata["lm_head"].data_ptr())
        self.vscratch = torch.empty(B.cass_verify_from_parts_scratch_bytes(self.desc), dtype=torch.uint8, device=self.device)
        torch.cuda.synchronize(self.device)
        B.cass_session_verify_from_parts(self.session, self._mv, self.vscratch)
        if drop_bf16:
            for lw in self.w["layers"]:
                for nm in ("wqkv", "wo", "wgu", "wd"):
                    lw[nm] = None
            self.w["lm_head"] = None
        return total

    def blob_bytes(self) -> int:
        return sum(sum(t.numel() for t in d.values()) for d in self.blobs["layers"]) + self.blobs["lm_head"].numel()

    def build_kv_codebook(self):
        B.cass_kv_build_codebook(self.session, self.n_prompt)

    # ------------------------------------------------------------------ decoding
    def next_tokens(self) -> torch.Tensor:
        """The token every sequence feeds into its next step ([batch], a copy)."""
        return self.toks[: self.batch * self._stride: self._stride].clone()

    def set_next_tokens(self, toks: torch.Tensor, non_blocking: bool = False):
        self.toks[: self.batch * self._stride: self._stride].copy_(toks, non_blocking=non_blocking)

    def _layout(self, gamma: int):
        """Moves the next input tokens to where a step with this gamma expects them: toks[b * (gamma + 1)]."""
        if self._stride != gamma + 1:
            nxt = self.toks[: self.batch * self._stride: self._stride].clone()
            self._stride = gamma + 1
            self.toks[: self.batch * self._stride: self._stride] = nxt

    def _spec_step(self, gamma: int):
        s = gamma + 1
        for i in range(gamma):
            B.cass_draft_step(self.session, self.toks[i:], self.toks[i + 1:], tok_stride=s)
        B.cass_verify(self.session, self.toks, gamma, self.targ)
        B.cass_accept(self.session, self.toks[1:], self.targ, gamma, self.n_acc, self.out_tokens, self.toks,
                      draft_stride=s, next_stride=s)

    def step(self, gamma: int):
        """One speculative step (gamma = 0: one plain autoregressive step) of every sequence.  Results stay on the
        device: n_acc[b] accepted drafts, out_tokens[b][0..n_acc[b]] emitted tokens, toks[b][0] the next input
        (arrays of gamma + 1 entries per sequence)."""
        self._layout(gamma)
        self._spec_step(gamma)

    def generate(self, n_tokens: int, gamma: int, use_graph: bool = False, sync_every: int = 1):
        """Emits at least n_tokens tokens per sequence after the prefill token.  Returns (tokens, StepStats): tokens
        is a list (batch 1) or a list of per-sequence lists."""
        out: list[list[int]] = [[] for _ in range(self.batch)]
        stats = StepStats()
        self._layout(gamma)
        if use_graph and gamma not in self._graphs:
            # capture needs a warm step and the captured step also executes nothing by itself: do both here
            self._spec_step(gamma)
            self._collect(out, stats)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                self._spec_step(gamma)
            self._graphs[gamma] = graph
        while min(len(o) for o in out) < n_tokens:
            if use_graph:
                self._graphs[gamma].replay()
            else:
                self._spec_step(gamma)
            self._collect(out, stats)
        return (out[0] if self.batch == 1 else out), stats

    def _collect(self, out, stats):
        s = self._stride
        acc = self.n_acc[: self.batch].tolist()
        toks = self.out_tokens[: self.batch * s].view(self.batch, s).tolist()
        for b, a in enumerate(acc):
            out[b].extend(toks[b][: a + 1])
            stats.accepted += a
            stats.emitted += a + 1
        stats.steps += 1

    def status(self) -> tuple[int, int]:
        return B.cass_session_status(self.session)

    def lens(self) -> list[int]:
        return B.cass_session_lens(self.session, self.batch)
