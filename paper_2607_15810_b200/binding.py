"""Thin ctypes binding over libquads.so: argument marshalling only.  Every step
of the path runs inside the library's CUDA kernels; torch is used for device
memory and the current stream.  Importing this module fails loudly when the
library has not been built (run `python -m paper_2607_15810_b200.build`)."""
import ctypes as C
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libquads.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError("libquads.so is missing: build it with `python -m paper_2607_15810_b200.build` "
                      "(there is no CPU fallback)")
lib = C.CDLL(_LIB_PATH)

QUADS_OK = 0
SF_LINEAR, SF_TILED = 0, 1

_p, _i32, _i64, _sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t


class MoEArgs(C.Structure):
    _fields_ = [
        ("T", _i32), ("H", _i32), ("I", _i32), ("E", _i32), ("topk", _i32), ("N", _i32),
        ("x", _p), ("router_logits", _p),
        ("w13_q", _p), ("w13_sf", _p), ("w13_gs", _p),
        ("w2_q", _p), ("w2_sf", _p), ("w2_gs", _p),
        ("rac_nsel_13", _i32), ("rac_nsel_2", _i32),
        ("a13_gs", _p), ("a2_gs", _p),
        ("renormalize", _i32),
        ("out", _p),
        ("topk_ids", _p), ("topk_w", _p), ("expert_offsets", _p), ("perm", _p),
        ("xq", _p), ("xsf", _p), ("rq", _p), ("rsf", _p), ("sel13", _p), ("a13_gs_out", _p),
        ("h_bf16", _p), ("hq", _p), ("hsf", _p), ("r2q", _p), ("r2sf", _p), ("sel2", _p),
        ("workspace", _p), ("workspace_bytes", _sz),
        ("operand_mode", _i32), ("w13_bf16", _p),
        ("expert_lo", _i32), ("expert_count", _i32), ("out_f32", _p),
    ]


lib.quads_status_string.restype = C.c_char_p
lib.quads_status_string.argtypes = [_i32]
lib.quads_sf_tiled_bytes.restype = _sz
lib.quads_sf_tiled_bytes.argtypes = [_i64, _i64]
lib.quads_quantize_workspace_bytes.restype = _sz
lib.quads_quantize_workspace_bytes.argtypes = []
lib.quads_fake_quant_workspace_bytes.restype = _sz
lib.quads_fake_quant_workspace_bytes.argtypes = [_i64]
lib.quads_moe_workspace_bytes.restype = _sz
lib.quads_moe_workspace_bytes.argtypes = [_i32] * 6
lib.quads_quantize_nvfp4.restype = _i32
lib.quads_quantize_nvfp4.argtypes = [_p, _i64, _i64, _i64, _p, _p, _p, _p, C.c_int, _p, _sz, _p]
lib.quads_fake_quant_weights.restype = _i32
lib.quads_fake_quant_weights.argtypes = [_p, _i64, _i64, _i64, _p, _p, _p, _p, C.c_int, _p, _sz, _p]
lib.quads_dequantize_nvfp4.restype = _i32
lib.quads_dequantize_nvfp4.argtypes = [_p, _p, _p, _i64, _i64, _i64, C.c_int, _p, _p]
lib.quads_fake_quant_activations.restype = _i32
lib.quads_fake_quant_activations.argtypes = [_p, _i64, _i64, _i64, _p, _p, _p, _p, _sz, _p]
lib.quads_fake_quant_weights_noalloc.restype = _i32
lib.quads_fake_quant_weights_noalloc.argtypes = [_p, _i64, _i64, _i64, _p, _p, _p, _p, C.c_int, _p]
lib.quads_moe_w4a4_rac.restype = _i32
lib.quads_moe_w4a4_rac.argtypes = [C.POINTER(MoEArgs), _p]
lib.quads_moe_async_status.restype = _i32
lib.quads_moe_async_status.argtypes = [_p, _p]
lib.quads_moe_set_kernel_timing.restype = _i32
lib.quads_moe_set_kernel_timing.argtypes = [_i32]
lib.quads_moe_last_kernel_ms.restype = _i32
lib.quads_moe_last_kernel_ms.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_float)]
lib.quads_last_launch_count.restype = _i32
lib.quads_last_launch_count.argtypes = []


class QuadsError(RuntimeError):
    def __init__(self, status):
        self.status = int(status)
        super().__init__(lib.quads_status_string(int(status)).decode())


def check(status):
    if status != QUADS_OK:
        raise QuadsError(status)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def sf_tiled_bytes(rows, K):
    return lib.quads_sf_tiled_bytes(rows, K)


def last_launch_count():
    return lib.quads_last_launch_count()


def _ws(nbytes, device):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def quantize_nvfp4(x, gs=None, sf_layout=SF_LINEAR, out=None, workspace=None):
    """x: bf16 CUDA tensor [rows, K] (row stride allowed).  Returns (q, sf, gs)."""
    assert x.dtype == torch.bfloat16 and x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    dev = x.device
    if out is None:
        q = torch.empty(rows, K // 2, dtype=torch.uint8, device=dev)
        n_sf = sf_tiled_bytes(rows, K) if sf_layout == SF_TILED else rows * (K // 16)
        sf = torch.empty(n_sf, dtype=torch.uint8, device=dev)
        if sf_layout == SF_LINEAR:
            sf = sf.view(rows, K // 16)
        gs_out = torch.empty(1, dtype=torch.float32, device=dev)
    else:
        q, sf, gs_out = out
    ws = workspace if workspace is not None else _ws(lib.quads_quantize_workspace_bytes(), dev)
    ld = x.stride(0) if rows > 1 else max(K, x.stride(0))
    check(lib.quads_quantize_nvfp4(_ptr(x), rows, K, ld, _ptr(gs), _ptr(q), _ptr(sf), _ptr(gs_out),
                                   sf_layout, _ptr(ws), ws.numel(), _stream()))
    return q, sf, gs_out


def dequantize_nvfp4(q, sf, gs, rows, K, sf_layout=SF_LINEAR, out=None):
    """q: u8 [n, rows, K/2]; sf: u8 per layout; gs: f32 [n].  Returns bf16 [n, rows, K]."""
    n = q.shape[0]
    if out is None:
        out = torch.empty(n, rows, K, dtype=torch.bfloat16, device=q.device)
    check(lib.quads_dequantize_nvfp4(_ptr(q), _ptr(sf), _ptr(gs), n, rows, K, sf_layout, _ptr(out), _stream()))
    return out


def fake_quant_activations(x, gs=None, out=None, workspace=None):
    """x: bf16 CUDA tensor [rows, K] (row stride allowed).  Returns (x_fq bf16 [rows, K], gs)."""
    assert x.dtype == torch.bfloat16 and x.is_cuda and x.dim() == 2 and x.stride(1) == 1
    rows, K = x.shape
    dev = x.device
    if out is None:
        x_fq = torch.empty(rows, K, dtype=torch.bfloat16, device=dev)
        gs_out = torch.empty(1, dtype=torch.float32, device=dev)
    else:
        x_fq, gs_out = out
    ws = workspace if workspace is not None else _ws(lib.quads_quantize_workspace_bytes(), dev)
    ld = x.stride(0) if rows > 1 else max(K, x.stride(0))
    check(lib.quads_fake_quant_activations(_ptr(x), rows, K, ld, _ptr(gs), _ptr(x_fq), _ptr(gs_out), _ptr(ws),
                                           ws.numel(), _stream()))
    return x_fq, gs_out


def fake_quant_weights(w, want_fq=True, want_pack=True, sf_layout=SF_LINEAR, out=None, workspace=None):
    """w: bf16 CUDA tensor [n, N, K] contiguous.  Returns dict(w_fq, q, sf, gs)."""
    assert w.dtype == torch.bfloat16 and w.is_cuda and w.dim() == 3 and w.is_contiguous()
    n, N, K = w.shape
    dev = w.device
    if out is None:
        w_fq = torch.empty_like(w) if want_fq else None
        q = torch.empty(n, N, K // 2, dtype=torch.uint8, device=dev) if want_pack else None
        if want_pack:
            per = sf_tiled_bytes(N, K) if sf_layout == SF_TILED else N * (K // 16)
            sf = torch.empty(n, per, dtype=torch.uint8, device=dev)
            if sf_layout == SF_LINEAR:
                sf = sf.view(n, N, K // 16)
        else:
            sf = None
        gs = torch.empty(n, dtype=torch.float32, device=dev)
    else:
        w_fq, q, sf, gs = out
    ws = workspace if workspace is not None else _ws(lib.quads_fake_quant_workspace_bytes(n), dev)
    check(lib.quads_fake_quant_weights(_ptr(w), n, N, K, _ptr(w_fq), _ptr(q), _ptr(sf), _ptr(gs), sf_layout,
                                       _ptr(ws), ws.numel(), _stream()))
    return dict(w_fq=w_fq, q=q, sf=sf, gs=gs)


NOALLOC_MAX_TENSORS = 4096


def fake_quant_weights_noalloc(w, out, sf_layout=SF_LINEAR, n_tensors=None):
    """Allocation-free fake-quant: for callers that may not allocate device
    memory (their memory belongs to a pool they do not own, or an allocation's
    implicit synchronisation is not allowed where they run).  `out` = (w_fq, q,
    sf, gs), all caller-allocated (any of the first three may be None); no
    workspace is passed and this wrapper creates no tensor.  `n_tensors`
    overrides the count taken from w's shape (used to probe the capacity
    check)."""
    n, N, K = w.shape
    w_fq, q, sf, gs = out
    check(lib.quads_fake_quant_weights_noalloc(_ptr(w), n if n_tensors is None else n_tensors, N, K, _ptr(w_fq),
                                               _ptr(q), _ptr(sf), _ptr(gs), sf_layout, _stream()))


def moe_workspace_bytes(T, H, I, E, topk, N=0):
    return lib.quads_moe_workspace_bytes(T, H, I, E, topk, N)


def moe_w4a4_rac(x, logits, w13, w2, topk, nsel13, nsel2, a2_gs, a13_gs=None, renormalize=True,
                 export=False, workspace=None, out=None, expert_range=None, out_f32=None):
    """MoE layer forward.  w13 / w2: dicts with q [E,rows,K/2], sf (tiled, [E,bytes]), gs [E] as
    produced by fake_quant_weights(..., sf_layout=SF_TILED).  Returns dict(out=bf16 [T,H], ...)."""
    T, H = x.shape
    E = logits.shape[1]
    I = w2["q"].shape[2] * 2
    dev = x.device
    A = T * topk
    a = MoEArgs()
    a.T, a.H, a.I, a.E, a.topk, a.N = T, H, I, E, topk, 0
    a.x, a.router_logits = _ptr(x), _ptr(logits)
    a.w13_q, a.w13_sf, a.w13_gs = _ptr(w13["q"]), _ptr(w13["sf"]), _ptr(w13["gs"])
    a.w2_q, a.w2_sf, a.w2_gs = _ptr(w2["q"]), _ptr(w2["sf"]), _ptr(w2["gs"])
    a.rac_nsel_13, a.rac_nsel_2 = nsel13, nsel2
    a.a13_gs, a.a2_gs = _ptr(a13_gs), _ptr(a2_gs)
    a.renormalize = 1 if renormalize else 0
    if expert_range is not None:            # w13 / w2 hold the experts lo .. hi-1 only; out_f32 gets their partial sum
        a.expert_lo, a.expert_count = expert_range[0], expert_range[1] - expert_range[0]
    res = {}
    res["out"] = out if out is not None else torch.empty(T, H, dtype=torch.bfloat16, device=dev)
    a.out = _ptr(res["out"])
    if out_f32 is not None:
        res["out_f32"] = out_f32
        a.out_f32 = _ptr(out_f32)
    if export:
        u8, i32, f32 = torch.uint8, torch.int32, torch.float32
        res["ids"] = torch.empty(T, topk, dtype=i32, device=dev)
        res["weights"] = torch.empty(T, topk, dtype=f32, device=dev)
        res["offsets"] = torch.empty(E + 1, dtype=i32, device=dev)
        res["perm"] = torch.empty(A, dtype=i32, device=dev)
        res["xq"] = torch.empty(T, H // 2, dtype=u8, device=dev)
        res["xsf"] = torch.empty(T, H // 16, dtype=u8, device=dev)
        res["rq"] = torch.zeros(T, H // 2, dtype=u8, device=dev)
        res["rsf"] = torch.zeros(T, H // 16, dtype=u8, device=dev)
        res["sel13"] = torch.empty(max(nsel13, 1), dtype=i32, device=dev)
        res["a13_gs"] = torch.empty(1, dtype=f32, device=dev)
        res["h"] = torch.empty(A, I, dtype=torch.bfloat16, device=dev)
        res["hq"] = torch.empty(A, I // 2, dtype=u8, device=dev)
        res["hsf"] = torch.empty(A, I // 16, dtype=u8, device=dev)
        res["r2q"] = torch.zeros(A, I // 2, dtype=u8, device=dev)
        res["r2sf"] = torch.zeros(A, I // 16, dtype=u8, device=dev)
        res["sel2"] = torch.empty(max(nsel2, 1), dtype=i32, device=dev)
        a.topk_ids, a.topk_w, a.expert_offsets, a.perm = map(_ptr, (res["ids"], res["weights"], res["offsets"], res["perm"]))
        a.xq, a.xsf, a.rq, a.rsf = map(_ptr, (res["xq"], res["xsf"], res["rq"], res["rsf"]))
        a.sel13, a.a13_gs_out = _ptr(res["sel13"]), _ptr(res["a13_gs"])
        a.h_bf16, a.hq, a.hsf = _ptr(res["h"]), _ptr(res["hq"]), _ptr(res["hsf"])
        a.r2q, a.r2sf, a.sel2 = _ptr(res["r2q"]), _ptr(res["r2sf"]), _ptr(res["sel2"])
    ws = workspace if workspace is not None else _ws(moe_workspace_bytes(T, H, I, E, topk), dev)
    a.workspace, a.workspace_bytes = _ptr(ws), ws.numel()
    check(lib.quads_moe_w4a4_rac(C.byref(a), _stream()))
    res["workspace"] = ws
    return res


def dense_w4a4_rac(x, w, nsel, a_gs=None, export=False, workspace=None):
    """Single projection out[T,N] = W X~.  w: dict(q [1,N,K/2] or [N,K/2], sf tiled, gs [1])."""
    T, K = x.shape
    N = w["q"].shape[-2]
    dev = x.device
    a = MoEArgs()
    a.T, a.H, a.I, a.E, a.topk, a.N = T, K, 0, 1, 1, N
    a.x = _ptr(x)
    a.w13_q, a.w13_sf, a.w13_gs = _ptr(w["q"]), _ptr(w["sf"]), _ptr(w["gs"])
    a.rac_nsel_13 = nsel
    a.a13_gs = _ptr(a_gs)
    res = {"out": torch.empty(T, N, dtype=torch.bfloat16, device=dev)}
    a.out = _ptr(res["out"])
    if export:
        u8 = torch.uint8
        res["xq"] = torch.empty(T, K // 2, dtype=u8, device=dev)
        res["xsf"] = torch.empty(T, K // 16, dtype=u8, device=dev)
        res["rq"] = torch.zeros(T, K // 2, dtype=u8, device=dev)
        res["rsf"] = torch.zeros(T, K // 16, dtype=u8, device=dev)
        res["sel13"] = torch.empty(max(nsel, 1), dtype=torch.int32, device=dev)
        res["a13_gs"] = torch.empty(1, dtype=torch.float32, device=dev)
        a.xq, a.xsf, a.rq, a.rsf = map(_ptr, (res["xq"], res["xsf"], res["rq"], res["rsf"]))
        a.sel13, a.a13_gs_out = _ptr(res["sel13"]), _ptr(res["a13_gs"])
    ws = workspace if workspace is not None else _ws(moe_workspace_bytes(T, K, 0, 1, 1, N), dev)
    a.workspace, a.workspace_bytes = _ptr(ws), ws.numel()
    check(lib.quads_moe_w4a4_rac(C.byref(a), _stream()))
    res["workspace"] = ws
    return res


W4A4, W4A16, W16A4, W16A16 = 0, 1, 2, 3


def dense_one_sided(x, mode, w=None, w_bf16=None, a_gs=None, export=False, workspace=None):
    """The one-sided rollout modes of the dense projection: mode = W4A16 (w: packed NVFP4 weight
    dict, x stays bf16) or W16A4 (w_bf16: bf16 [N, K] weight, x quantized online and decoded).
    Returns dict(out=bf16 [T, N], ...)."""
    T, K = x.shape
    N = w["q"].shape[-2] if mode == W4A16 else w_bf16.shape[0]
    assert mode in (W4A16, W16A4, W16A16)
    dev = x.device
    a = MoEArgs()
    a.T, a.H, a.I, a.E, a.topk, a.N = T, K, 0, 1, 1, N
    a.x = _ptr(x)
    a.operand_mode = mode
    if mode == W4A16:
        a.w13_q, a.w13_sf, a.w13_gs = _ptr(w["q"]), _ptr(w["sf"]), _ptr(w["gs"])
    else:
        a.w13_bf16 = _ptr(w_bf16)
        a.a13_gs = _ptr(a_gs) if mode == W16A4 else None
    res = {"out": torch.empty(T, N, dtype=torch.bfloat16, device=dev)}
    a.out = _ptr(res["out"])
    if export and mode == W16A4:
        res["xq"] = torch.empty(T, K // 2, dtype=torch.uint8, device=dev)
        res["xsf"] = torch.empty(T, K // 16, dtype=torch.uint8, device=dev)
        res["a13_gs"] = torch.empty(1, dtype=torch.float32, device=dev)
        a.xq, a.xsf, a.a13_gs_out = _ptr(res["xq"]), _ptr(res["xsf"]), _ptr(res["a13_gs"])
    ws = workspace if workspace is not None else _ws(moe_workspace_bytes(T, K, 0, 1, 1, N), dev)
    a.workspace, a.workspace_bytes = _ptr(ws), ws.numel()
    check(lib.quads_moe_w4a4_rac(C.byref(a), _stream()))
    res["workspace"] = ws
    return res


def moe_async_status(workspace):
    return lib.quads_moe_async_status(_ptr(workspace), _stream())


def moe_set_kernel_timing(enable):
    check(lib.quads_moe_set_kernel_timing(1 if enable else 0))


def moe_last_kernel_ms():
    """(gemm1_ms, gemm2_ms) of the most recent timed MoE call."""
    a, b = C.c_float(), C.c_float()
    check(lib.quads_moe_last_kernel_ms(C.byref(a), C.byref(b)))
    return a.value, b.value


lib.quads_moe_set_stage_trace.restype = _i32
lib.quads_moe_set_stage_trace.argtypes = [_i32]
lib.quads_moe_get_stage_trace.restype = _i32
lib.quads_moe_get_stage_trace.argtypes = [C.POINTER(C.c_char_p), C.POINTER(C.c_float), _i32]


def moe_set_stage_trace(enable):
    check(lib.quads_moe_set_stage_trace(1 if enable else 0))


def moe_get_stage_trace():
    """[(stage name, ms)] of the most recent traced MoE call."""
    names = (C.c_char_p * 40)()
    ms = (C.c_float * 40)()
    n = lib.quads_moe_get_stage_trace(names, ms, 40)
    return [(names[i].decode(), ms[i]) for i in range(n)]


lib.quads_fp4_pipe_probe.restype = _i32
lib.quads_fp4_pipe_probe.argtypes = [_i32, _i32, _p, _sz, _p, C.POINTER(C.c_double), _p]
lib.quads_fp4_pipe_probe_operand_bytes.restype = _sz
lib.quads_fp4_pipe_probe_operand_bytes.argtypes = []


def fp4_pipe_probe(mode, k_steps, operands, status_word):
    """Enqueue the tensor-pipe probe; returns the floating-point operations of the launch."""
    flop = C.c_double()
    check(lib.quads_fp4_pipe_probe(mode, k_steps, _ptr(operands), operands.numel() * operands.element_size(),
                                   _ptr(status_word), C.byref(flop), _stream()))
    return flop.value


lib.quads_rac_channel_scores.restype = _i32
lib.quads_rac_channel_scores.argtypes = [_p, _i64, _i64, _p, _p, _p, _sz, _p]
lib.quads_rac_channel_scores_workspace_bytes.restype = _sz
lib.quads_rac_channel_scores_workspace_bytes.argtypes = [_i64, _i64]
lib.quads_mismatch_norms.restype = _i32
lib.quads_mismatch_norms.argtypes = [_p, _p, _i64, _p, _p, _sz, _p]
lib.quads_mismatch_norms_workspace_bytes.restype = _sz
lib.quads_mismatch_norms_workspace_bytes.argtypes = []


def rac_channel_scores(x, gs=None, workspace=None):
    """Squared channel scores of Eq. channel-score: float64 [H] (device)."""
    T, H = x.shape
    scores = torch.empty(H, dtype=torch.float64, device=x.device)
    ws = workspace if workspace is not None else _ws(lib.quads_rac_channel_scores_workspace_bytes(T, H), x.device)
    check(lib.quads_rac_channel_scores(_ptr(x), T, H, _ptr(gs), _ptr(scores), _ptr(ws), ws.numel(), _stream()))
    return scores


def mismatch_norms(a, b, workspace=None):
    """float64 [3] (device): ||a - b||^2, ||a||^2, ||b||^2 over two bf16 tensors of equal size."""
    assert a.dtype == torch.bfloat16 and b.dtype == torch.bfloat16 and a.numel() == b.numel()
    assert a.is_contiguous() and b.is_contiguous()
    out = torch.empty(3, dtype=torch.float64, device=a.device)
    ws = workspace if workspace is not None else _ws(lib.quads_mismatch_norms_workspace_bytes(), a.device)
    check(lib.quads_mismatch_norms(_ptr(a), _ptr(b), a.numel(), _ptr(out), _ptr(ws), ws.numel(), _stream()))
    return out


class MoEFp8Args(C.Structure):
    _fields_ = [
        ("T", _i32), ("H", _i32), ("I", _i32), ("E", _i32), ("topk", _i32),
        ("x", _p), ("router_logits", _p),
        ("w13_q", _p), ("w13_atoms", _p), ("w2_q", _p), ("w2_atoms", _p),
        ("renormalize", _i32),
        ("out", _p),
        ("topk_ids", _p), ("perm", _p), ("xq", _p), ("xexp", _p), ("h_bf16", _p), ("hq", _p), ("hexp", _p),
        ("workspace", _p), ("workspace_bytes", _sz),
    ]


lib.quads_fp8_quantize_weights.restype = _i32
lib.quads_fp8_quantize_weights.argtypes = [_p, _i64, _i64, _i64, _p, _p, _p, _p]
lib.quads_moe_fp8_w8a8.restype = _i32
lib.quads_moe_fp8_w8a8.argtypes = [C.POINTER(MoEFp8Args), _p]
lib.quads_moe_fp8_workspace_bytes.restype = _sz
lib.quads_moe_fp8_workspace_bytes.argtypes = [_i32] * 5


def fp8_quantize_weights(w):
    """w: bf16 CUDA [n, N, K] -> dict(q u8 [n, N, K], exps u8 [n, N/128, K/128], atoms u8 [n, N/128, K/128, 512])."""
    assert w.dtype == torch.bfloat16 and w.is_cuda and w.dim() == 3 and w.is_contiguous()
    n, N, K = w.shape
    dev = w.device
    q = torch.empty(n, N, K, dtype=torch.uint8, device=dev)
    exps = torch.empty(n, N // 128, K // 128, dtype=torch.uint8, device=dev)
    atoms = torch.empty(n, N // 128, K // 128, 512, dtype=torch.uint8, device=dev)
    check(lib.quads_fp8_quantize_weights(_ptr(w), n, N, K, _ptr(q), _ptr(exps), _ptr(atoms), _stream()))
    return dict(q=q, exps=exps, atoms=atoms)


def moe_fp8_workspace_bytes(T, H, I, E, topk):
    return lib.quads_moe_fp8_workspace_bytes(T, H, I, E, topk)


def moe_fp8_w8a8(x, logits, w13, w2, topk, renormalize=True, export=False, workspace=None, out=None):
    """FP8 W8A8 MoE layer (comparison path).  w13 / w2: dicts from fp8_quantize_weights."""
    T, H = x.shape
    E = logits.shape[1]
    I = w2["q"].shape[2]
    dev = x.device
    A = T * topk
    a = MoEFp8Args()
    a.T, a.H, a.I, a.E, a.topk = T, H, I, E, topk
    a.x, a.router_logits = _ptr(x), _ptr(logits)
    a.w13_q, a.w13_atoms, a.w2_q, a.w2_atoms = _ptr(w13["q"]), _ptr(w13["atoms"]), _ptr(w2["q"]), _ptr(w2["atoms"])
    a.renormalize = 1 if renormalize else 0
    res = {"out": out if out is not None else torch.empty(T, H, dtype=torch.bfloat16, device=dev)}
    a.out = _ptr(res["out"])
    if export:
        u8 = torch.uint8
        res["ids"] = torch.empty(T, topk, dtype=torch.int32, device=dev)
        res["perm"] = torch.empty(A, dtype=torch.int32, device=dev)
        res["xq"] = torch.empty(T, H, dtype=u8, device=dev)
        res["xexp"] = torch.empty(T, H // 128, dtype=u8, device=dev)
        res["h"] = torch.empty(A, I, dtype=torch.bfloat16, device=dev)
        res["hq"] = torch.empty(A, I, dtype=u8, device=dev)
        res["hexp"] = torch.empty(A, I // 128, dtype=u8, device=dev)
        a.topk_ids, a.perm, a.xq, a.xexp = map(_ptr, (res["ids"], res["perm"], res["xq"], res["xexp"]))
        a.h_bf16, a.hq, a.hexp = map(_ptr, (res["h"], res["hq"], res["hexp"]))
    ws = workspace if workspace is not None else _ws(moe_fp8_workspace_bytes(T, H, I, E, topk), dev)
    a.workspace, a.workspace_bytes = _ptr(ws), ws.numel()
    check(lib.quads_moe_fp8_w8a8(C.byref(a), _stream()))
    res["workspace"] = ws
    return res
