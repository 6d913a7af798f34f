"""Python face of the context API: owns the device arenas (torch tensors) and forwards every call to libspec.so.

Marshalling only: sizes come from spec_query_sizes, addresses from spec_tensor, and each step method is one C call.
"""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from . import binding as B
from .binding import T


def make_spec_config(cfg: dict, *, draft_kind: str = "none", k_max: int = 3, max_batch: int = 4, kv_num_blocks: int = 64,
                     max_blocks_per_seq: int = 16, kv_block_tokens: int = 16, kv_layer_pools: int | None = None,
                     seed: int = 0, draft_d_ffn: int | None = None, ngram_n: int = 3, draft_greedy: bool = False,
                     draft_vocab: int = 0, kv_fp8=None, w_fp8: bool = False) -> B.spec_config:
    """kv_fp8: None for a cache in the model's dtype, or (k_scale, v_scale) for the 8-bit e4m3 cache.
    w_fp8: the target's projections and LM head in e4m3 with per-row scales (a reduced-precision mode)."""
    sc = B.spec_config()
    sc.struct_size, sc.abi_version = C.sizeof(B.spec_config), B.SPEC_ABI_VERSION
    for name in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "n_experts",
                 "experts_top_k", "d_expert_ffn"):
        setattr(sc, name, int(cfg.get(name, 0)))
    sc.rms_eps, sc.rope_theta = float(cfg["rms_eps"]), float(cfg["rope_theta"])
    sc.dtype = B.SPEC_DTYPE_F32 if cfg["dtype"] == "f32" else B.SPEC_DTYPE_BF16
    sc.draft_kind = {"none": B.SPEC_DRAFT_NONE, "eagle3": B.SPEC_DRAFT_EAGLE3, "mtp": B.SPEC_DRAFT_MTP, "ngram": B.SPEC_DRAFT_NGRAM}[draft_kind]
    sc.draft_d_ffn = int(draft_d_ffn if draft_d_ffn is not None else (cfg["d_ffn"] or 4 * cfg["d_model"])) if draft_kind in ("eagle3", "mtp") else 0
    sc.ngram_n = int(ngram_n) if draft_kind == "ngram" else 0
    sc.draft_greedy = 1 if draft_greedy else 0
    sc.draft_vocab = int(draft_vocab) if draft_kind == "eagle3" else 0
    if kv_fp8:
        sc.kv_dtype, sc.kv_scale_k, sc.kv_scale_v = B.SPEC_KV_E4M3, float(kv_fp8[0]), float(kv_fp8[1])
    sc.weight_dtype = B.SPEC_W_E4M3 if (w_fp8 or cfg.get("w_fp8")) else B.SPEC_W_MODEL
    taps = tuple(cfg.get("tap_layers", ())) if draft_kind == "eagle3" else ()
    sc.n_taps = len(taps)
    for i, t in enumerate(taps):
        sc.tap_layers[i] = int(t)
    sc.k_max, sc.max_batch = int(k_max), int(max_batch)
    sc.kv_block_tokens, sc.kv_num_blocks, sc.max_blocks_per_seq = int(kv_block_tokens), int(kv_num_blocks), int(max_blocks_per_seq)
    sc.kv_layer_pools = int(kv_layer_pools if kv_layer_pools is not None else cfg["n_layers"])
    sc.temperature, sc.seed = float(cfg.get("temperature", 1.0)), int(seed)
    return sc


def stack_gate_up(gate, up):
    """[.., F, d] gate and up -> the library's stacked layout [.., 2F, d]: 256-row groups of 128 gate rows followed by
    the matching 128 up rows.  numpy arrays or torch tensors."""
    if hasattr(gate, "data_ptr"):
        F, d = gate.shape[-2:]
        lead = tuple(gate.shape[:-2])
        g = gate.reshape(lead + (F // 128, 128, d))
        u = up.reshape(lead + (F // 128, 128, d))
        return torch.cat([g, u], dim=-2).reshape(lead + (2 * F, d))
    gate, up = np.asarray(gate), np.asarray(up)
    F, d = gate.shape[-2:]
    lead = gate.shape[:-2]
    g = gate.reshape(lead + (F // 128, 128, d))
    u = up.reshape(lead + (F // 128, 128, d))
    return np.concatenate([g, u], axis=-2).reshape(lead + (2 * F, d))


def unstack_gate_up(gu):
    """Inverse of stack_gate_up: returns (gate, up)."""
    gu = np.asarray(gu)
    F2, d = gu.shape[-2:]
    lead = gu.shape[:-2]
    t = gu.reshape(lead + (F2 // 256, 256, d))
    return t[..., :128, :].reshape(lead + (F2 // 2, d)), t[..., 128:, :].reshape(lead + (F2 // 2, d))


class SpecStep:
    """One context over arenas allocated here.  Methods mirror the C entry points one to one."""

    def __init__(self, sc: B.spec_config, device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("the speculation step runs on a CUDA device only (no CPU fallback)")
        self.lib = B.lib()
        self.sc = sc
        self.device = torch.device(device)
        self.tdtype = torch.float32 if sc.dtype == B.SPEC_DTYPE_F32 else torch.bfloat16
        sizes = B.spec_sizes()
        B._check(self.lib.spec_query_sizes(C.byref(sc), C.byref(sizes)), "spec_query_sizes")
        self.sizes = sizes
        self.arenas = {}
        bufs = B.spec_buffers()
        for name in ("weights", "draft_weights", "kv", "draft_kv", "workspace", "state"):
            n = getattr(sizes, name + "_bytes")
            t = torch.zeros(max(n, 256), dtype=torch.uint8, device=self.device) if name in ("state", "workspace") \
                else torch.empty(max(n, 256), dtype=torch.uint8, device=self.device)
            self.arenas[name] = t
            setattr(bufs, name, t.data_ptr())
        self.bufs = bufs
        h = C.c_void_p()
        B._check(self.lib.spec_create(C.byref(sc), C.byref(bufs), C.byref(h)), "spec_create")
        self.ctx = h
        self.B = 0

    def close(self):
        if self.ctx:
            self.lib.spec_destroy(self.ctx)
            self.ctx = None

    # ---- tensors -------------------------------------------------------------------------------------------
    def tensor(self, name: str, layer: int = 0, dtype=None, shape=None) -> torch.Tensor:
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        B._check(self.lib.spec_tensor(self.ctx, T[name], layer, C.byref(ptr), C.byref(nbytes)), f"spec_tensor({name})")
        for a in self.arenas.values():
            off = ptr.value - a.data_ptr()
            if 0 <= off < a.numel():
                raw = a[off : off + nbytes.value]
                break
        else:
            raise RuntimeError("tensor outside the arenas")
        if dtype is None:
            return raw
        t = raw.view(dtype)
        if shape is not None:
            n = int(np.prod(shape))
            t = t[:n].view(*shape)
        return t

    def put(self, name: str, layer: int, array, dtype=None):
        """Writes a host array into a weight / cache tensor (cast to the tensor's storage type)."""
        dtype = dtype or self.tdtype
        src = torch.from_numpy(np.ascontiguousarray(array)).to(self.device).to(dtype).reshape(-1)
        dst = self.tensor(name, layer, dtype)
        assert src.numel() <= dst.numel(), (name, src.numel(), dst.numel())
        dst[: src.numel()].copy_(src)

    def put_projection(self, name: str, layer: int, array):
        """A projection weight [rows][K]: stored as it is, or - in a context with 8-bit weights - as e4m3 codes with one
        scale per row, quantised on the device by the library (spec_quantize_rows) from the 16-bit values."""
        if self.sc.weight_dtype != B.SPEC_W_E4M3:
            return self.put(name, layer, array)
        w = array if torch.is_tensor(array) else torch.from_numpy(np.ascontiguousarray(array))
        w = w.to(self.device).to(torch.bfloat16)
        w = w.reshape(-1, w.shape[-1]).contiguous()                # experts [E][rows][K]: every row of every expert has its scale
        codes = self.tensor(name, layer, torch.uint8)
        scales = self.tensor(name + "_SCALE", layer, torch.float32)
        assert codes.numel() == w.numel() and scales.numel() == w.shape[0], (name, codes.numel(), w.numel(), scales.numel())
        B.spec_quantize_rows(w, codes.view(w.shape), scales)
        torch.cuda.synchronize()

    def load_target_weights(self, W: dict):
        f32 = torch.float32
        self.put("EMBED", 0, W["embed"])
        self.put_projection("LM_HEAD", 0, W["lm_head"])
        self.put("FINAL_NORM", 0, W["final_norm"], f32)
        for l, lw in enumerate(W["layers"]):
            self.put("ATTN_NORM", l, lw["attn_norm"], f32)
            self.put_projection("WQKV", l, lw["wqkv"])
            self.put_projection("WO", l, lw["wo"])
            self.put("MLP_NORM", l, lw["mlp_norm"], f32)
            if "router" in lw:
                self.put("ROUTER", l, lw["router"])
                self.put_projection("EXPERTS_GATEUP", l, stack_gate_up(lw["experts_gate"], lw["experts_up"]))
                self.put_projection("EXPERTS_DOWN", l, lw["experts_down"])
            else:
                self.put_projection("WGATEUP", l, stack_gate_up(lw["wgate"], lw["wup"]))
                self.put_projection("WDOWN", l, lw["wdown"])

    def load_draft_weights(self, H: dict):
        f32 = torch.float32
        self.put("D_NORM_E", 0, H["norm_e"], f32)
        self.put("D_NORM_G", 0, H["norm_g"], f32)
        self.put("D_MLP_NORM", 0, H["mlp_norm"], f32)
        self.put("D_WQKV", 0, H["wqkv"])
        self.put("D_WO", 0, H["wo"])
        self.put("D_WGATEUP", 0, stack_gate_up(H["wgate"], H["wup"]))
        self.put("D_WDOWN", 0, H["wdown"])
        if self.sc.draft_kind == B.SPEC_DRAFT_EAGLE3:
            self.put("D_WFC", 0, H["wfc"])
            self.put("D_NORM_F", 0, H["norm_f"], f32)
            self.put("D_LM_HEAD", 0, H["lm_head"])
            if self.sc.draft_vocab:
                assert H["lm_head"].shape[0] == self.sc.draft_vocab and len(H["d2t"]) == self.sc.draft_vocab
                self.put("D_D2T", 0, np.asarray(H["d2t"], np.int32), torch.int32)
        else:
            self.put("D_WPROJ", 0, H["wproj"])
            self.put("D_ATTN_NORM", 0, H["attn_norm"], f32)

    # ---- the step ------------------------------------------------------------------------------------------------
    def seq_init(self, seq_len, last_token, free_stack, stream=None):
        sl = np.ascontiguousarray(seq_len, np.int32)
        lt = np.ascontiguousarray(last_token, np.int32)
        fs = np.ascontiguousarray(free_stack, np.int32)
        assert fs.shape[0] == self.sc.kv_num_blocks
        B._check(self.lib.spec_seq_init(self.ctx, sl.shape[0], sl.ctypes.data, lt.ctypes.data, fs.ctypes.data,
                                        B._stream(stream)), "spec_seq_init")
        self.B = sl.shape[0]

    def seq_replace(self, slots, seq_len, last_token, stream=None):
        sl = np.ascontiguousarray(slots, np.int32)
        ln = np.ascontiguousarray(seq_len, np.int32)
        lt = np.ascontiguousarray(last_token, np.int32)
        assert sl.shape == ln.shape == lt.shape
        B._check(self.lib.spec_seq_replace(self.ctx, sl.shape[0], sl.ctypes.data, ln.ctypes.data, lt.ctypes.data,
                                           B._stream(stream)), "spec_seq_replace")

    def seq_compact(self, keep_slots, stream=None):
        """Shrinks the batch to the listed (ascending) slots; everything else is retired.  Updates self.B."""
        ks = np.ascontiguousarray(keep_slots, np.int32)
        B._check(self.lib.spec_seq_compact(self.ctx, ks.shape[0], ks.ctypes.data if ks.shape[0] else None, B._stream(stream)), "spec_seq_compact")
        self.B = int(ks.shape[0])

    def capture_step(self, k, with_draft=True):
        """Captures draft(k) -> verify(k) -> reject_sample(k) -> kv_commit() into a CUDA graph (the step functions only
        enqueue work, and the step counter and all sequence state live on the device) and returns the graph; `replay()` it
        on the current stream in place of the four calls.  Worth it when the batch is thin and the step is a chain of
        hundreds of short kernels.  The graph is tied to the current batch size: capture again after seq_init or
        seq_compact.  A plain step with the same k must have run before (lazy one-time initialisation happens outside a
        capture), and no forced commit or caller-supplied drafts can go through a captured step."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            if with_draft:
                self.draft(k)
            self.verify(k)
            self.reject_sample(k)
            self.kv_commit()
        torch.cuda.current_stream().wait_stream(side)
        return graph

    def draft(self, k, stream=None):
        B._check(self.lib.spec_draft(self.ctx, k, B._stream(stream)), "spec_draft")

    def verify(self, k, draft_tokens=None, stream=None):
        B._check(self.lib.spec_verify(self.ctx, k, B._ptr(draft_tokens), B._stream(stream)), "spec_verify")

    def reject_sample(self, k, draft_logits=None, stream=None):
        B._check(self.lib.spec_reject_sample(self.ctx, k, B._ptr(draft_logits), B._stream(stream)), "spec_reject_sample")

    def kv_commit(self, force_n=None, force_token=None, stream=None):
        B._check(self.lib.spec_kv_commit(self.ctx, B._ptr(force_n), B._ptr(force_token), B._stream(stream)), "spec_kv_commit")

    def status(self, stream=None) -> B.spec_step_report:
        rep = B.spec_step_report()
        B._check(self.lib.spec_get_status(self.ctx, C.byref(rep), B._stream(stream)), "spec_get_status")
        return rep

    def set_timing(self, mask: int):
        B._check(self.lib.spec_set_timing(self.ctx, mask), "spec_set_timing")

    def get_timing(self, stream=None) -> B.spec_timing:
        t = B.spec_timing()
        B._check(self.lib.spec_get_timing(self.ctx, C.byref(t), B._stream(stream)), "spec_get_timing")
        return t

    # ---- typed views of step results -----------------------------------------------------------------------------
    def logits(self, k):
        return self.tensor("LOGITS", 0, torch.float32, (self.B, k + 1, self.sc.vocab))

    def draft_logits(self, k):
        return self.tensor("DRAFT_LOGITS", 0, torch.float32, (self.B, k, self.sc.draft_vocab or self.sc.vocab))

    def out_tokens(self, k):
        return self.tensor("OUT_TOKENS", 0, torch.int32, (self.B, k + 1))

    def out_logp(self, k):
        return self.tensor("OUT_LOGP", 0, torch.float32, (self.B, k + 1))

    def n_emitted(self):
        return self.tensor("N_EMITTED", 0, torch.int32, (self.B,))

    def draft_tokens(self):
        return self.tensor("DRAFT_TOKENS", 0, torch.int32, (self.sc.max_batch, max(self.sc.k_max, 1)))[: self.B]

    def seq_len(self):
        return self.tensor("SEQ_LEN", 0, torch.int32, (self.B,))

    def block_table(self):
        return self.tensor("BLOCK_TABLE", 0, torch.int32, (self.sc.max_batch, self.sc.max_blocks_per_seq))[: self.B]

    def kv_pool(self, which: str, pool: int = 0):
        sc = self.sc
        dt = torch.uint8 if sc.kv_dtype == B.SPEC_KV_E4M3 else self.tdtype           # e4m3 codes are handed out as bytes
        return self.tensor(which, pool, dt, (sc.kv_num_blocks, sc.n_kv_heads, sc.kv_block_tokens, sc.head_dim))

    def kv_pool_values(self, which: str, pool: int = 0):
        """The pool as fp32 values (codes times the scale for the 8-bit cache)."""
        sc = self.sc
        p = self.kv_pool(which, pool)
        if sc.kv_dtype != B.SPEC_KV_E4M3:
            return p.float()
        scale = sc.kv_scale_k if which.endswith("_K") else sc.kv_scale_v
        return p.view(torch.float8_e4m3fn).float() * scale
