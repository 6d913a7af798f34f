"""Thin ctypes binding of libspec.so: the same names as include/spec.h, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; torch is used for device memory and streams.  There is
no CPU fallback: importing works without a GPU (so that symbols can be checked), any compute call without the
library or without a device raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspec.so")

SPEC_ABI_VERSION = 6
SPEC_DTYPE_BF16, SPEC_DTYPE_F32 = 0, 1
SPEC_KV_MODEL, SPEC_KV_E4M3 = 0, 1
SPEC_W_MODEL, SPEC_W_E4M3 = 0, 1
SPEC_DRAFT_NONE, SPEC_DRAFT_EAGLE3, SPEC_DRAFT_MTP, SPEC_DRAFT_NGRAM = 0, 1, 2, 3

STATUS_NAMES = {0: "SPEC_OK", -1: "SPEC_ERR_INVALID_ARG", -2: "SPEC_ERR_SHAPE", -3: "SPEC_ERR_UNSUPPORTED",
                -4: "SPEC_ERR_STATE", -5: "SPEC_ERR_CUDA", -16: "SPEC_ERR_KV_EXHAUSTED",
                -17: "SPEC_ERR_TOKEN_RANGE", -18: "SPEC_ERR_BAD_PROB", -19: "SPEC_ERR_TIMEOUT",
                -20: "SPEC_ERR_EP_CAPACITY"}

# tensor ids (spec.h)
T = dict(EMBED=0, LM_HEAD=1, FINAL_NORM=2, ATTN_NORM=3, WQKV=4, WO=5, MLP_NORM=6, WGATEUP=7, WDOWN=8, ROUTER=9,
         EXPERTS_GATEUP=10, EXPERTS_DOWN=11, LM_HEAD_SCALE=16, WQKV_SCALE=17, WO_SCALE=18, WGATEUP_SCALE=19, WDOWN_SCALE=20, EXPERTS_GATEUP_SCALE=21, EXPERTS_DOWN_SCALE=22,
         D_WFC=32, D_WPROJ=33, D_NORM_E=34, D_NORM_G=35, D_NORM_F=36, D_ATTN_NORM=37, D_WQKV=38, D_WO=39,
         D_MLP_NORM=40, D_WGATEUP=41, D_WDOWN=42, D_LM_HEAD=43, D_D2T=44,
         KV_K=64, KV_V=65, DRAFT_KV_K=66, DRAFT_KV_V=67,
         SEQ_LEN=96, LAST_TOKEN=97, BLOCK_TABLE=98, FREE_STACK=99, FREE_TOP=100, DRAFT_TOKENS=101, OUT_TOKENS=102,
         N_EMITTED=103, STATUS=104, STEP=105, TOKEN_HISTORY=106, OUT_LOGP=107,
         LOGITS=128, DRAFT_LOGITS=129, ROW_STATS=130, DRAFT_ROW_STATS=131, TAPS=132, HIDDEN=133, MOE_LOGITS=134, MOE_IDS=135, MOE_WTS=136,
         ACT_CODES=137, ACT_SCALES=138, MOE_INV=139)


class SpecError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")
        self.code = code


class spec_config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("abi_version", C.c_uint32),
                ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("n_experts", C.c_int32), ("experts_top_k", C.c_int32), ("d_expert_ffn", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("dtype", C.c_int32), ("draft_kind", C.c_int32), ("draft_d_ffn", C.c_int32),
                ("n_taps", C.c_int32), ("tap_layers", C.c_int32 * 3),
                ("k_max", C.c_int32), ("max_batch", C.c_int32), ("kv_block_tokens", C.c_int32),
                ("kv_num_blocks", C.c_int32), ("max_blocks_per_seq", C.c_int32), ("kv_layer_pools", C.c_int32),
                ("temperature", C.c_float), ("seed", C.c_uint64), ("ngram_n", C.c_int32), ("draft_greedy", C.c_int32), ("draft_vocab", C.c_int32), ("kv_dtype", C.c_int32),
                ("kv_scale_k", C.c_float), ("kv_scale_v", C.c_float), ("weight_dtype", C.c_int32)]


class spec_sizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("weights_bytes", "draft_weights_bytes", "kv_bytes", "draft_kv_bytes",
                                          "workspace_bytes", "state_bytes")]


class spec_buffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("weights", "draft_weights", "kv", "draft_kv", "workspace", "state")]


class spec_timing(C.Structure):
    _fields_ = [("ms", C.c_float * 4), ("passes", C.c_int32 * 4), ("dropped", C.c_int32)]


class spec_ep_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("ep_size", "ep_rank", "n_experts", "top_k", "d", "d_expert_ffn", "max_rows", "cap_rows")]


class spec_ep_sizes(C.Structure):
    _fields_ = [("window_bytes", C.c_size_t), ("scratch_bytes", C.c_size_t)]


EP_T = dict(IDS=0, WTS=1, COUNTS=2, RECV_OFF=3, RECV_TOTAL=4, EXPERT_OUT=5, RECV_ROWS=6)


class spec_step_report(C.Structure):
    _fields_ = [("device_status", C.c_int32), ("device_detail", C.c_int32), ("steps", C.c_int64),
                ("emitted_tokens", C.c_int64), ("accepted_drafts", C.c_int64)]


_vp, _i, _f, _u32, _u64, _sz = C.c_void_p, C.c_int, C.c_float, C.c_uint32, C.c_uint64, C.c_size_t

# name -> (restype, argtypes): every symbol include/spec.h declares
SIGNATURES = {
    "spec_query_sizes": (_i, [C.POINTER(spec_config), C.POINTER(spec_sizes)]),
    "spec_create": (_i, [C.POINTER(spec_config), C.POINTER(spec_buffers), C.POINTER(_vp)]),
    "spec_destroy": (_i, [_vp]),
    "spec_tensor": (_i, [_vp, _i, _i, C.POINTER(_vp), C.POINTER(_sz)]),
    "spec_seq_init": (_i, [_vp, _i, _vp, _vp, _vp, _vp]),
    "spec_seq_replace": (_i, [_vp, _i, _vp, _vp, _vp, _vp]),
    "spec_seq_compact": (_i, [_vp, _i, _vp, _vp]),
    "spec_draft": (_i, [_vp, _i, _vp]),
    "spec_verify": (_i, [_vp, _i, _vp, _vp]),
    "spec_reject_sample": (_i, [_vp, _i, _vp, _vp]),
    "spec_kv_commit": (_i, [_vp, _vp, _vp, _vp]),
    "spec_get_status": (_i, [_vp, C.POINTER(spec_step_report), _vp]),
    "spec_last_error": (C.c_char_p, [_vp]),
    "spec_softmax_rows": (_i, [_i, _i, _vp, _f, _vp, _vp, _vp]),
    "spec_sample_rows": (_i, [_i, _i, _vp, _u64, _u32, _u32, _u32, _vp, _vp, _vp]),
    "spec_reject_sample_probs": (_i, [_i, _i, _i, _vp, _vp, _vp, _u64, _u32, _vp, _vp, _vp, _vp]),
    "spec_reject_sample_logits": (_i, [_i, _i, _i, _vp, _vp, _vp, _vp, _vp, _f, _u64, _u32, _vp, _vp, _vp, _vp]),
    "spec_uniforms": (_i, [_u64, _u32, _u32, _i, _i, _vp, _vp]),
    "spec_quantize_rows": (_i, [_i, _i, _vp, _vp, _vp, _vp]),
    "spec_gemm": (_i, [_i, _i, _i, _vp, _vp, _vp, _i, _i, _i, _vp]),
    "spec_gemm_e4m3": (_i, [_i, _i, _i, _vp, _vp, _vp, _vp, _vp, _i, _i, _vp]),
    "spec_attention": (_i, [_i, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp, _sz, _vp]),
    "spec_attention_scratch_bytes": (_sz, [_i, _i, _i, _i, _i, _i]),
    "spec_attention_noalloc": (_i, [_i, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _i, _vp]),
    "spec_set_timing": (_i, [_vp, _u32]),
    "spec_get_timing": (_i, [_vp, C.POINTER(spec_timing), _vp]),
    "spec_selftest_bounded_wait": (_i, [_vp, _vp, _vp]),
    "spec_ep_query_sizes": (_i, [C.POINTER(spec_ep_config), C.POINTER(spec_ep_sizes)]),
    "spec_ep_tensor": (_i, [C.POINTER(spec_ep_config), _vp, _vp, _i, C.POINTER(_vp), C.POINTER(_sz)]),
    "spec_ep_route": (_i, [C.POINTER(spec_ep_config), _vp, _vp, _i, _vp, _vp, _vp]),
    "spec_ep_route_e4m3": (_i, [C.POINTER(spec_ep_config), _vp, _vp, _i, _vp, _vp, _vp]),
    "spec_ep_experts": (_i, [C.POINTER(spec_ep_config), C.POINTER(_vp), _vp, _vp, _vp, _vp, _vp]),
    "spec_ep_experts_e4m3": (_i, [C.POINTER(spec_ep_config), C.POINTER(_vp), _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "spec_ep_combine": (_i, [C.POINTER(spec_ep_config), C.POINTER(_vp), _i, _vp, _vp]),
    "spec_ipc_export": (_i, [_vp, _vp, C.POINTER(_u64)]),
    "spec_ipc_open": (_i, [_vp, C.POINTER(_vp)]),
    "spec_ipc_close": (_i, [_vp]),
    "spec_launch_count": (C.c_int64, []),
    "spec_version": (C.c_char_p, []),
}

_lib = None


def lib():
    """Loads libspec.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_26779_b200.build` "
                               "(the library is the only implementation; there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / None / int."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous()
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(code, where):
    if code != 0:
        raise SpecError(code, where)


# ---- stateless entry points ------------------------------------------------------------------------------------

def spec_softmax_rows(logits, temperature=1.0, stats=None, probs=None, stream=None):
    V = logits.shape[-1]
    rows = logits.numel() // V
    _check(lib().spec_softmax_rows(rows, V, _ptr(logits), float(temperature), _ptr(stats), _ptr(probs), _stream(stream)),
           "spec_softmax_rows")


def spec_sample_rows(probs, seed, step, slot, stream_tag, tokens, status=None, stream=None):
    rows, V = probs.shape
    _check(lib().spec_sample_rows(rows, V, _ptr(probs), seed, step, slot, stream_tag, _ptr(tokens), _ptr(status),
                                  _stream(stream)), "spec_sample_rows")


def spec_reject_sample_probs(p, q, draft, seed, step, out_tokens, n_emitted, status=None, stream=None):
    B, kp1, V = p.shape
    _check(lib().spec_reject_sample_probs(B, kp1 - 1, V, _ptr(p), _ptr(q), _ptr(draft), seed, step, _ptr(out_tokens),
                                          _ptr(n_emitted), _ptr(status), _stream(stream)), "spec_reject_sample_probs")


def spec_reject_sample_logits(p_logits, p_stats, q_logits, q_stats, draft, temperature, seed, step, out_tokens,
                              n_emitted, status=None, stream=None):
    B, kp1, V = p_logits.shape
    _check(lib().spec_reject_sample_logits(B, kp1 - 1, V, _ptr(p_logits), _ptr(p_stats), _ptr(q_logits), _ptr(q_stats),
                                           _ptr(draft), float(temperature), seed, step, _ptr(out_tokens),
                                           _ptr(n_emitted), _ptr(status), _stream(stream)), "spec_reject_sample_logits")


def spec_uniforms(seed, step, stream_tag, u, stream=None):
    n_seq, n_slots = u.shape
    _check(lib().spec_uniforms(seed, step, stream_tag, n_seq, n_slots, _ptr(u), _stream(stream)), "spec_uniforms")


def spec_quantize_rows(x, codes, scales, stream=None):
    rows, K = x.shape
    _check(lib().spec_quantize_rows(rows, K, _ptr(x), _ptr(codes), _ptr(scales), _stream(stream)), "spec_quantize_rows")


def spec_gemm(A, W, Cout, accumulate=False, stream=None):
    import torch
    M, K = A.shape
    N = W.shape[0]
    din = SPEC_DTYPE_F32 if A.dtype == torch.float32 else SPEC_DTYPE_BF16
    dout = SPEC_DTYPE_F32 if Cout.dtype == torch.float32 else SPEC_DTYPE_BF16
    _check(lib().spec_gemm(M, N, K, _ptr(A), _ptr(W), _ptr(Cout), din, dout, int(accumulate), _stream(stream)),
           "spec_gemm")


def spec_gemm_e4m3(a8, a_scale, w8, w_scale, Cout, accumulate=False, stream=None):
    import torch
    M, K = a8.shape
    N = w8.shape[0]
    out_dt = SPEC_DTYPE_BF16 if Cout.dtype == torch.bfloat16 else SPEC_DTYPE_F32
    _check(lib().spec_gemm_e4m3(M, N, K, _ptr(a8), _ptr(a_scale), _ptr(w8), _ptr(w_scale), _ptr(Cout), out_dt, int(accumulate), _stream(stream)),
           "spec_gemm_e4m3")


def spec_attention_scratch_bytes(B, R, Hq, Hkv, dh, max_kv_len):
    return lib().spec_attention_scratch_bytes(B, R, Hq, Hkv, dh, max_kv_len)


def spec_attention(q, k_pool, v_pool, block_table, seq_len, out, scratch, stream=None):
    import torch
    B, R, Hq, dh = q.shape
    _, Hkv, bt, _ = k_pool.shape
    dt = SPEC_DTYPE_F32 if q.dtype == torch.float32 else SPEC_DTYPE_BF16
    _check(lib().spec_attention(B, R, Hq, Hkv, dh, bt, block_table.shape[1], _ptr(q), _ptr(k_pool), _ptr(v_pool),
                                _ptr(block_table), _ptr(seq_len), _ptr(out), dt, _ptr(scratch),
                                scratch.numel() * scratch.element_size(), _stream(stream)), "spec_attention")


def spec_attention_noalloc(q, k_pool, v_pool, block_table, seq_len, out, stream=None):
    """spec_attention with the library's built-in 32 MiB scratch: for callers that must not allocate device memory.
    Raises SpecError(SPEC_ERR_SHAPE) when the shapes need more scratch than that."""
    import torch
    B, R, Hq, dh = q.shape
    _, Hkv, bt, _ = k_pool.shape
    dt = SPEC_DTYPE_F32 if q.dtype == torch.float32 else SPEC_DTYPE_BF16
    _check(lib().spec_attention_noalloc(B, R, Hq, Hkv, dh, bt, block_table.shape[1], _ptr(q), _ptr(k_pool), _ptr(v_pool),
                                        _ptr(block_table), _ptr(seq_len), _ptr(out), dt, _stream(stream)),
           "spec_attention_noalloc")


def spec_ep_query_sizes(cfg):
    out = spec_ep_sizes()
    _check(lib().spec_ep_query_sizes(C.byref(cfg), C.byref(out)), "spec_ep_query_sizes")
    return out


def spec_ep_tensor(cfg, window, scratch, tensor_id):
    """(device address, bytes) of one piece of a window / scratch."""
    p, n = _vp(), _sz()
    _check(lib().spec_ep_tensor(C.byref(cfg), _ptr(window), _ptr(scratch), tensor_id, C.byref(p), C.byref(n)), "spec_ep_tensor")
    return p.value, n.value


def _peer_array(peer_windows):
    return (_vp * len(peer_windows))(*[_ptr(w) for w in peer_windows])


def spec_ep_route(cfg, window, scratch, M, h, router_w, stream=None):
    _check(lib().spec_ep_route(C.byref(cfg), _ptr(window), _ptr(scratch), M, _ptr(h), _ptr(router_w), _stream(stream)), "spec_ep_route")


def spec_ep_route_e4m3(cfg, window, scratch, M, h, router_w, stream=None):
    _check(lib().spec_ep_route_e4m3(C.byref(cfg), _ptr(window), _ptr(scratch), M, _ptr(h), _ptr(router_w), _stream(stream)), "spec_ep_route_e4m3")


def spec_ep_experts(cfg, peer_windows, scratch, w_gateup, w_down, status=None, stream=None):
    _check(lib().spec_ep_experts(C.byref(cfg), _peer_array(peer_windows), _ptr(scratch), _ptr(w_gateup), _ptr(w_down),
                                 _ptr(status), _stream(stream)), "spec_ep_experts")


def spec_ep_experts_e4m3(cfg, peer_windows, scratch, w_gateup, w_gateup_scale, w_down, w_down_scale, status=None, stream=None):
    _check(lib().spec_ep_experts_e4m3(C.byref(cfg), _peer_array(peer_windows), _ptr(scratch), _ptr(w_gateup), _ptr(w_gateup_scale),
                                      _ptr(w_down), _ptr(w_down_scale), _ptr(status), _stream(stream)), "spec_ep_experts_e4m3")


def spec_ep_combine(cfg, peer_windows, M, x, stream=None):
    _check(lib().spec_ep_combine(C.byref(cfg), _peer_array(peer_windows), M, _ptr(x), _stream(stream)), "spec_ep_combine")


def spec_ipc_export(dev_ptr):
    """(64-byte handle, offset of dev_ptr inside its allocation)."""
    h = (C.c_ubyte * 64)()
    off = _u64()
    _check(lib().spec_ipc_export(_ptr(dev_ptr), h, C.byref(off)), "spec_ipc_export")
    return bytes(h), off.value


def spec_ipc_open(handle):
    buf = (C.c_ubyte * 64).from_buffer_copy(handle)
    p = _vp()
    _check(lib().spec_ipc_open(buf, C.byref(p)), "spec_ipc_open")
    return p.value


def spec_ipc_close(base):
    _check(lib().spec_ipc_close(base), "spec_ipc_close")


def spec_version():
    return lib().spec_version().decode()


def spec_launch_count():
    return int(lib().spec_launch_count())
