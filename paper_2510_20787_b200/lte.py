"""Thin Python binding over the C-ABI library ``liblte.so`` (argument marshalling only).

Every function takes CUDA ``torch`` tensors (device memory and the current stream are all PyTorch
is used for), checks dtype / contiguity, and passes raw pointers to the entry point of the same name
declared in ``include/lte.h``.  There is no fallback: if the library is missing or a call fails, an
exception is raised.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblte.so")
_lib = None

F32, BF16 = 0, 1
OP_SCORES, OP_SELECT, OP_PREFILL, OP_DECODE, OP_BWD, OP_CHUNK, OP_STATS, OP_CHUNK_STREAM = range(8)
CHUNK_STREAMING = 1
BWD_CNN_INPUT_GRAD = 1

EXPORTS = ["lte_device_status", "lte_workspace_bytes", "lte_strerror", "lte_scores", "lte_select", "lte_cache_score", "lte_attn_prefill",
           "lte_cache_bytes", "lte_cache_init", "lte_attn_decode", "lte_attn_prefill_chunk", "lte_attn_bwd", "lte_attn_bwd_static",
           "lte_sparsity_stats", "lte_lambda_update", "lte_cache_score_unrope", "lte_selftest_per_device", "lte_select_rule", "lte_attn_colsum", "lte_attn_prefill_chunk_ex"]
STATIC_SCRATCH_BYTES = 8 << 20


class LteShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T", ctypes.c_int32), ("d", ctypes.c_int32),
                ("W", ctypes.c_int32), ("R", ctypes.c_int32), ("sink", ctypes.c_int32),
                ("tau", ctypes.c_float), ("softmax_scale", ctypes.c_float), ("dtype", ctypes.c_int32),
                ("group", ctypes.c_int32)]


class LteConv(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("kernel", ctypes.c_int32), ("dilation", ctypes.c_int32),
                ("w", ctypes.c_void_p), ("bias", ctypes.c_void_p)]


class LteError(RuntimeError):
    def __init__(self, fn, status):
        self.status = status
        super().__init__("%s failed: %d (%s)" % (fn, status, lib().lte_strerror(status).decode()))


def lib():
    """Load ``liblte.so`` (built by ``python -m paper_2510_20787_b200.build``); raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("liblte.so is not built: run `python -m paper_2510_20787_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.lte_strerror.restype = ctypes.c_char_p
        L.lte_strerror.argtypes = [ctypes.c_int]
        L.lte_workspace_bytes.restype = ctypes.c_size_t
        L.lte_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        L.lte_device_status.restype = ctypes.c_int
        L.lte_device_status.argtypes = []
        L.lte_cache_bytes.restype = ctypes.c_size_t
        L.lte_cache_bytes.argtypes = [ctypes.c_void_p]
        vp = ctypes.c_void_p
        L.lte_scores.argtypes = [vp] * 7 + [ctypes.c_size_t, vp]
        L.lte_select.argtypes = [vp] * 6 + [ctypes.c_size_t, vp]
        L.lte_attn_prefill.argtypes = [vp] * 9 + [ctypes.c_size_t, vp]
        L.lte_cache_init.argtypes = [vp] * 9
        L.lte_attn_decode.argtypes = [vp] * 9
        L.lte_cache_score.argtypes = [vp] * 4 + [ctypes.c_size_t, vp]
        L.lte_cache_score_unrope.argtypes = [vp] * 5 + [ctypes.c_int32, vp, ctypes.c_size_t, vp]
        L.lte_sparsity_stats.argtypes = [vp] * 6 + [ctypes.c_size_t, vp]
        L.lte_lambda_update.argtypes = [ctypes.c_int32, vp, vp, vp, ctypes.c_int64, vp]
        L.lte_attn_prefill_chunk.argtypes = [vp] * 3 + [ctypes.c_int32] + [vp] * 6 + [ctypes.c_size_t, vp]
        L.lte_attn_prefill_chunk_ex.argtypes = [vp] * 3 + [ctypes.c_int32] + [vp] * 5 + [ctypes.c_uint32, vp, ctypes.c_size_t, vp]
        L.lte_attn_bwd.argtypes = [vp] * 17 + [ctypes.c_uint32, vp, ctypes.c_size_t, vp]
        L.lte_attn_bwd_static.argtypes = [vp] * 17 + [ctypes.c_uint32, vp]
        L.lte_selftest_per_device.argtypes = [ctypes.c_int]
        L.lte_select_rule.argtypes = [vp, ctypes.c_int] + [vp] * 5 + [ctypes.c_size_t, vp]
        L.lte_attn_colsum.argtypes = [vp] * 8
        for name in EXPORTS:
            if name not in ("lte_strerror", "lte_workspace_bytes", "lte_cache_bytes", "lte_device_status"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _dt(t):
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("q/k/v must be float32 or bfloat16")


def shape(B, H, T, d, W, R, dtype, sink=0, tau=0.5, softmax_scale=0.0, group=1):
    """H key/value heads; with group > 1 (grouped-query attention) q, o and lse have H * group heads."""
    return LteShape(B, H, T, d, W, R, sink, tau, softmax_scale, dtype, group)


def conv(w, bias=None):
    """w: CUDA fp32 [H, K, 2d]; bias: CUDA fp32 [H] or None."""
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
    assert bias is None or (bias.is_cuda and bias.dtype == torch.float32 and bias.is_contiguous())
    c = LteConv(1, w.shape[1], 1, w.data_ptr(), 0 if bias is None else bias.data_ptr())
    c._keep = (w, bias)          # the struct only holds raw pointers: keep the tensors alive with it
    return c


def conv_stack(wl, wout, bl=None, bout=None):
    """The paper's three-layer scorer for lte_scores: wl = [wl0 [H,d,3,2d], wl1 [H,d/2,3,d], wl2 [H,d/4,3,d/2]],
    wout [H,d/4]; bl = three bias tensors [H,c] or None, bout [H] or None.  All CUDA fp32.  The tensors are packed
    into the two buffers the C struct carries."""
    assert len(wl) == 3 and all(t.is_cuda and t.dtype == torch.float32 for t in list(wl) + [wout])
    w = torch.cat([t.contiguous().reshape(-1) for t in list(wl) + [wout]]).contiguous()
    b = None
    if bl is not None or bout is not None:
        H = wout.shape[0]
        parts = [(bl[i] if bl is not None and bl[i] is not None else torch.zeros((H, wl[i].shape[1]), device=w.device))
                 for i in range(3)]
        parts.append(bout if bout is not None else torch.zeros((H,), device=w.device))
        b = torch.cat([t.to(torch.float32).contiguous().reshape(-1) for t in parts]).contiguous()
    c = LteConv(3, 3, 2, w.data_ptr(), 0 if b is None else b.data_ptr())
    c._keep = (w, b)
    return c


def _ptr(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    if dtype is not None:
        assert t.dtype == dtype, "expected %s, got %s" % (dtype, t.dtype)
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _check(fn, status):
    if status != 0:
        raise LteError(fn, status)


def lte_device_status():
    """0, or LTE_ERR_DEVICE_STATUS (-6) if a kernel gave up on a bounded wait since the last call."""
    return int(lib().lte_device_status())


def lte_workspace_bytes(op, s, c=None):
    return int(lib().lte_workspace_bytes(op, ctypes.addressof(s), None if c is None else ctypes.addressof(c)))


def lte_scores(s, c, k, v, z=None, r=None, ws=None):
    """k, v [B,H,T,d] -> z [B,H,T] fp32 (and r = sigmoid(z) if a tensor is given).  ws: a uint8 workspace tensor of
    lte_workspace_bytes(OP_SCORES, s, c) bytes (allocated here when None and the call wants one; False = none)."""
    if z is None:
        z = torch.empty((s.B, s.H, s.T), dtype=torch.float32, device=k.device)
    if ws is None:
        n = lte_workspace_bytes(OP_SCORES, s, c)
        ws = torch.empty(n, dtype=torch.uint8, device=k.device) if n > 0 else False
    wp, wn = (None, 0) if ws is False else (_ptr(ws, torch.uint8), ws.numel())
    _check("lte_scores", lib().lte_scores(ctypes.addressof(s), ctypes.addressof(c), _ptr(k), _ptr(v),
                                          _ptr(z, torch.float32), _ptr(r, torch.float32), wp, wn, _stream()))
    return z


def lte_select(s, z, idx=None, cnt=None, ncand=None):
    """z [B,H,T] fp32 -> idx [B,H,R] int32 ascending (-1 unused), cnt [B,H] int32."""
    dev = z.device
    if idx is None:
        idx = torch.empty((s.B, s.H, s.R), dtype=torch.int32, device=dev)
    if cnt is None:
        cnt = torch.empty((s.B, s.H), dtype=torch.int32, device=dev)
    _check("lte_select", lib().lte_select(ctypes.addressof(s), _ptr(z, torch.float32), _ptr(idx, torch.int32),
                                          _ptr(cnt, torch.int32), _ptr(ncand, torch.int32), None, 0, _stream()))
    return idx, cnt


RULE_LEARNED, RULE_UNIFORM, RULE_ACCUM_ATTN = 0, 1, 2


def lte_select_rule(s, rule, score=None, idx=None, cnt=None, ncand=None, device=None):
    """lte_select under one of the rules: RULE_LEARNED (score = z), RULE_UNIFORM (no score), RULE_ACCUM_ATTN (score = the
    accumulated attention of lte_attn_colsum)."""
    dev = score.device if score is not None else (device or torch.device("cuda"))
    if idx is None:
        idx = torch.empty((s.B, s.H, s.R), dtype=torch.int32, device=dev)
    if cnt is None:
        cnt = torch.empty((s.B, s.H), dtype=torch.int32, device=dev)
    _check("lte_select_rule", lib().lte_select_rule(ctypes.addressof(s), int(rule), _ptr(score, torch.float32), _ptr(idx, torch.int32),
                                                    _ptr(cnt, torch.int32), _ptr(ncand, torch.int32), None, 0, _stream()))
    return idx, cnt


def lte_attn_colsum(s, q, k, lse, idx, cnt, a=None):
    """Accumulated attention a [B,H,T] fp32 of every key under the attention lte_attn_prefill ran with this list."""
    if a is None:
        a = torch.empty((s.B, s.H, s.T), dtype=torch.float32, device=q.device)
    _check("lte_attn_colsum", lib().lte_attn_colsum(ctypes.addressof(s), _ptr(q), _ptr(k), _ptr(lse, torch.float32),
                                                    _ptr(idx, torch.int32), _ptr(cnt, torch.int32), _ptr(a, torch.float32), _stream()))
    return a


def lte_attn_prefill(s, q, k, v, idx, cnt, o=None, lse=None, ws=None):
    """q [B,H*group,T,d], k, v [B,H,T,d], retained list -> o [B,H*group,T,d], lse [B,H*group,T] fp32.
    ws: uint8 tensor of lte_workspace_bytes(OP_PREFILL, s) bytes (the retained rows are compacted into it and fetched
    as tiles), allocated here when None; False: no workspace (the kernels gather the retained rows themselves)."""
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((s.B, s.H * max(s.group, 1), s.T), dtype=torch.float32, device=q.device)
    if ws is None:
        need = lte_workspace_bytes(OP_PREFILL, s, None)
        ws = torch.empty(need, dtype=torch.uint8, device=q.device) if need > 0 else False
    wp, wn = (None, 0) if ws is False else (_ptr(ws), ws.numel())
    _check("lte_attn_prefill", lib().lte_attn_prefill(ctypes.addressof(s), _ptr(q), _ptr(k), _ptr(v),
                                                      _ptr(idx, torch.int32), _ptr(cnt, torch.int32), _ptr(o),
                                                      _ptr(lse, torch.float32), wp, wn, _stream()))
    return o, lse


def lte_cache_bytes(s):
    return int(lib().lte_cache_bytes(ctypes.addressof(s)))


def lte_cache_init(s, c, k=None, v=None, z=None, idx=None, cnt=None, cache=None):
    """Decode cache holding the state after the T-token prompt (T = 0: empty cache)."""
    if cache is None:
        dev = k.device if k is not None else torch.device("cuda")
        cache = torch.empty(lte_cache_bytes(s), dtype=torch.uint8, device=dev)
    _check("lte_cache_init", lib().lte_cache_init(ctypes.addressof(s), ctypes.addressof(c), _ptr(k), _ptr(v),
                                                  _ptr(z), _ptr(idx), _ptr(cnt), _ptr(cache), _stream()))
    return cache


def lte_attn_decode(s, c, cache, q1, k1, v1, o1=None, lse1=None):
    """One decode step: q1 [B,H*group,d], k1, v1 [B,H,d] -> o1 [B,H*group,d], lse1 [B,H*group]; the cache is
    updated in place."""
    if o1 is None:
        o1 = torch.empty_like(q1)
    if lse1 is None:
        lse1 = torch.empty((s.B, s.H * max(s.group, 1)), dtype=torch.float32, device=q1.device)
    _check("lte_attn_decode", lib().lte_attn_decode(ctypes.addressof(s), ctypes.addressof(c), _ptr(cache),
                                                    _ptr(q1), _ptr(k1), _ptr(v1), _ptr(o1),
                                                    _ptr(lse1, torch.float32), _stream()))
    return o1, lse1


def lte_attn_prefill_chunk(s, c, cache, n_past, q, k, v, o=None, lse=None, ws=None, streaming=False):
    """Chunked prefill on top of a cache that holds n_past tokens: q [B,H*group,T,d], k, v [B,H,T,d] (T = s.T new
    tokens) -> o, lse of the chunk's queries; the cache is advanced to n_past + T tokens in place.  ws: uint8 tensor of
    lte_workspace_bytes(OP_CHUNK or OP_CHUNK_STREAM, s, c) bytes, allocated here when None.  streaming=True: the
    token-by-token reading (what decode steps compute, also where the cap binds)."""
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((s.B, s.H * max(s.group, 1), s.T), dtype=torch.float32, device=q.device)
    if ws is None:
        ws = torch.empty(max(lte_workspace_bytes(OP_CHUNK_STREAM if streaming else OP_CHUNK, s, c), 256), dtype=torch.uint8, device=q.device)
    _check("lte_attn_prefill_chunk", lib().lte_attn_prefill_chunk_ex(ctypes.addressof(s), ctypes.addressof(c), _ptr(cache),
                                                                     ctypes.c_int32(int(n_past)), _ptr(q), _ptr(k), _ptr(v),
                                                                     _ptr(o), _ptr(lse, torch.float32), CHUNK_STREAMING if streaming else 0,
                                                                     _ptr(ws), ws.numel(), _stream()))
    return o, lse


class LteLambdaCfg(ctypes.Structure):
    _fields_ = [("period", ctypes.c_int32), ("cap", ctypes.c_float), ("alpha", ctypes.c_float), ("band", ctypes.c_float),
                ("floor", ctypes.c_float), ("max", ctypes.c_float)]


def lte_sparsity_stats(s, z, lam=None, ws=None):
    """Eq. 7 statistics: z [B,H,T] -> count [H] (batch mean of tokens above the threshold), penalty [1]."""
    count = torch.empty((s.H,), dtype=torch.float32, device=z.device)
    penalty = torch.empty((1,), dtype=torch.float32, device=z.device)
    if ws is None:
        ws = torch.empty(max(lte_workspace_bytes(OP_STATS, s, None), 256), dtype=torch.uint8, device=z.device)
    _check("lte_sparsity_stats", lib().lte_sparsity_stats(ctypes.addressof(s), _ptr(z, torch.float32), _ptr(lam, torch.float32),
                                                          _ptr(count), _ptr(penalty), _ptr(ws), ws.numel(), _stream()))
    return count, penalty


def lte_lambda_update(lam, cbar, count, step, cfg=None, group=None):
    """Algorithm 1's feedback step on host tensors (float32, contiguous, updated in place).  When torch.distributed is
    initialised the counts are averaged over the ranks of `group` first, so that all ranks take the same decision."""
    import torch.distributed as dist
    assert lam.device.type == "cpu" and cbar.device.type == "cpu" and lam.dtype == torch.float32 and cbar.dtype == torch.float32
    count = count.detach().to("cpu", torch.float32).contiguous().clone()
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(count, group=group)
        count /= dist.get_world_size(group)
    _check("lte_lambda_update", lib().lte_lambda_update(lam.numel(), lam.data_ptr(), cbar.data_ptr(), count.data_ptr(), int(step),
                                                        ctypes.addressof(cfg) if cfg is not None else None))
    return lam, cbar


def lte_cache_score(s, c, cache, ws=None):
    """Three-layer stack only: score the ring tokens whose receptive field is complete (call at least every W - 13
    decode steps).  ws: uint8 tensor of lte_workspace_bytes(OP_DECODE, s, c) bytes, allocated here when None."""
    if ws is None:
        ws = torch.empty(max(lte_workspace_bytes(OP_DECODE, s, c), 256), dtype=torch.uint8, device=cache.device)
    _check("lte_cache_score", lib().lte_cache_score(ctypes.addressof(s), ctypes.addressof(c), _ptr(cache), _ptr(ws),
                                                    ws.numel(), _stream()))


def lte_cache_score_unrope(s, c, cache, rope_cos, rope_sin, ws=None):
    """lte_cache_score for a cache that holds rotated keys: rope_cos, rope_sin [positions, d/2] fp32 on the device."""
    if ws is None:
        ws = torch.empty(max(lte_workspace_bytes(OP_DECODE, s, c), 256), dtype=torch.uint8, device=cache.device)
    _check("lte_cache_score_unrope", lib().lte_cache_score_unrope(ctypes.addressof(s), ctypes.addressof(c), _ptr(cache),
                                                                  _ptr(rope_cos, torch.float32), _ptr(rope_sin, torch.float32),
                                                                  int(rope_cos.shape[0]), _ptr(ws), ws.numel(), _stream()))


def lte_attn_bwd(s, c, q, k, v, o, lse, dO, z, idx, cnt, lam=None, flags=BWD_CNN_INPUT_GRAD, want_dbias=True,
                 ws=None):
    """Backward with the straight-through surrogate -> dq, dk, dv, dw [H,K,2d], dbias [H] (or None).  With the
    three-layer stack (conv_stack) dw and dbias are flat, packed like the parameters: use unpack_stack_grads."""
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    if c.n_layers == 3:
        d = s.d
        dw = torch.empty((s.H * (d * 3 * 2 * d + (d // 2) * 3 * d + (d // 4) * 3 * (d // 2) + d // 4),), dtype=torch.float32, device=q.device)
        db = torch.empty((s.H * (d + d // 2 + d // 4 + 1),), dtype=torch.float32, device=q.device) if want_dbias else None
    else:
        dw = torch.empty((s.H, c.kernel, 2 * s.d), dtype=torch.float32, device=q.device)
        db = torch.empty((s.H,), dtype=torch.float32, device=q.device) if want_dbias else None
    need = lte_workspace_bytes(OP_BWD, s, c)
    if ws is None:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=q.device)
    _check("lte_attn_bwd", lib().lte_attn_bwd(
        ctypes.addressof(s), ctypes.addressof(c), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse, torch.float32),
        _ptr(dO), _ptr(z, torch.float32), _ptr(idx, torch.int32), _ptr(cnt, torch.int32),
        _ptr(lam, torch.float32), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dw), _ptr(db), flags, _ptr(ws),
        ws.numel(), _stream()))
    return dq, dk, dv, dw, db


def unpack_stack_grads(H, d, dw, db=None):
    """Flat gradients of the three-layer stack -> (dwl [3 tensors [H,c_out,3,c_in]], dwout [H,d/4], dbl [3] or None,
    dbout [H] or None), the shapes conv_stack takes."""
    ch = [2 * d, d, d // 2, d // 4]
    dwl, off = [], 0
    for l in range(3):
        n = H * ch[l + 1] * 3 * ch[l]
        dwl.append(dw[off:off + n].view(H, ch[l + 1], 3, ch[l])); off += n
    dwout = dw[off:off + H * ch[3]].view(H, ch[3])
    if db is None:
        return dwl, dwout, None, None
    dbl, off = [], 0
    for l in range(3):
        dbl.append(db[off:off + H * ch[l + 1]].view(H, ch[l + 1])); off += H * ch[l + 1]
    return dwl, dwout, dbl, db[off:off + H]


def lte_attn_bwd_static(s, c, q, k, v, o, lse, dO, z, idx, cnt, lam=None, flags=BWD_CNN_INPUT_GRAD, outs=None):
    """lte_attn_bwd with the library's built-in scratch array instead of a workspace: for callers that must not
    allocate device memory.  ``outs`` = (dq, dk, dv, dw, dbias) preallocated by the caller makes the whole call
    allocation-free; when omitted they are created here for convenience.  Shapes needing more scratch than
    STATIC_SCRATCH_BYTES raise LteError (status -3)."""
    if outs is None:
        outs = (torch.empty_like(q), torch.empty_like(k), torch.empty_like(v),
                torch.empty((s.H, c.kernel, 2 * s.d), dtype=torch.float32, device=q.device),
                torch.empty((s.H,), dtype=torch.float32, device=q.device))
    dq, dk, dv, dw, db = outs
    _check("lte_attn_bwd_static", lib().lte_attn_bwd_static(
        ctypes.addressof(s), ctypes.addressof(c), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse, torch.float32),
        _ptr(dO), _ptr(z, torch.float32), _ptr(idx, torch.int32), _ptr(cnt, torch.int32),
        _ptr(lam, torch.float32), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dw), _ptr(db), flags, _stream()))
    return dq, dk, dv, dw, db
