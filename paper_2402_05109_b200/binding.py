"""ctypes binding of include/hydra.h.  Names follow the C ABI; arguments are torch CUDA tensors."""
import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libhydra.so")
if not os.path.exists(LIB_PATH):
    raise ImportError("libhydra.so is not built: run `python -m paper_2402_05109_b200.build` (needs nvcc)")
lib = C.CDLL(LIB_PATH)


class HydraError(RuntimeError):
    pass


class ModelCfgC(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("dtype", C.c_int), ("max_batch", C.c_int),
                ("max_seq", C.c_int), ("kv_planes", C.c_int)]


class HeadCfgC(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_heads", "n_mlp_layers", "prefix_attn", "has_bias", "medusa")]


class TreeCfgC(C.Structure):
    _fields_ = [("n_rows", C.c_int), ("parent", C.POINTER(C.c_int32))]


_PP = C.POINTER(C.c_void_p)


class WeightsC(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", _PP), ("wqkv", _PP), ("wo", _PP), ("ffn_norm", _PP), ("w_gate_up", _PP), ("w_down", _PP),
                ("head_w1", _PP), ("head_b1", _PP), ("head_wr", _PP), ("head_br", _PP)] + \
               [(n, C.c_void_p) for n in ("pfx_attn_norm", "pfx_wqkv", "pfx_wo", "pfx_ffn_norm", "pfx_w_gate_up",
                                           "pfx_w_down")]


_vp, _i, _sz = C.c_void_p, C.c_int, C.c_size_t
lib.hydra_workspace_bytes.restype = _sz
lib.hydra_workspace_bytes.argtypes = [C.POINTER(ModelCfgC), C.POINTER(HeadCfgC), C.POINTER(TreeCfgC)]
lib.hydra_create.argtypes = [C.POINTER(_vp), C.POINTER(ModelCfgC), C.POINTER(HeadCfgC), C.POINTER(TreeCfgC),
                             C.POINTER(WeightsC), _vp, _sz]
lib.hydra_destroy.argtypes = [_vp]
lib.hydra_prefill.argtypes = [_vp, _i, _vp, C.POINTER(C.c_int32), _vp]
lib.hydra_draft.argtypes = [_vp, _vp, _vp]
lib.hydra_verify.argtypes = [_vp, _vp, _vp, _vp, _vp]
lib.hydra_accept_compact.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.hydra_step.argtypes = [_vp, _vp, _vp, _vp]
lib.hydra_set_plant.argtypes = [_vp, _vp]
lib.hydra_set_acceptance.argtypes = [_vp, _i, C.c_float, C.c_float, C.c_float, _vp]
lib.hydra_get_buffer.argtypes = [_vp, _i, C.POINTER(_vp), C.POINTER(_sz)]
lib.hydra_poll_status.argtypes = [_vp, _vp]
lib.hydra_launch_count.restype = C.c_longlong
lib.hydra_launch_count.argtypes = [_vp]
lib.hydra_set_gemm_mode.argtypes = [_vp, _i]
lib.hydra_set_step_graph.argtypes = [_vp, _i]
lib.hydra_set_timing.argtypes = [_vp, _i]
lib.hydra_get_timing.argtypes = [_vp, _i, C.POINTER(C.c_double), C.POINTER(C.c_longlong), C.POINTER(C.c_double)]
lib.hydra_status_str.restype = C.c_char_p
lib.hydra_status_str.argtypes = [_i]
lib.hydra_last_error.restype = C.c_char_p
lib.hydra_gemm_partial_floats.restype = _sz
lib.hydra_gemm_partial_floats.argtypes = [_i] * 5
lib.hydra_gemm.argtypes = [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp]
lib.hydra_gemm_noalloc.argtypes = [_vp, _vp, _vp, _i, _i, _i, _vp, _vp]
lib.hydra_gemm_bounded_wait_probe.argtypes = [_vp, _vp, _vp, _i, _i, _i, _i, C.c_uint, _vp, _vp, _vp]
lib.hydra_attention_scratch_bytes.restype = _sz
lib.hydra_attention_scratch_bytes.argtypes = [_i] * 5
lib.hydra_tree_attention.argtypes = [_vp] * 8 + [_i] * 8 + [_vp, _vp]

BUF = dict(LEN=0, ROOT_TOK=1, H_TREE=2, H_NEW=3, KV_BASE=4, KV_PREFIX=5, TREE_MASK=6, TREE_TOK=7, AMAX=8,
           HEAD_LOGITS=9, N_NEW=10, H_PRIME=11, STATUS=12, PASS_BITS=13)
_BUF_DTYPE = dict(LEN=torch.int32, ROOT_TOK=torch.int32, H_TREE=torch.float32, H_NEW=torch.float32,
                  TREE_MASK=torch.int64, TREE_TOK=torch.int32, AMAX=torch.int32, HEAD_LOGITS=torch.float32,
                  N_NEW=torch.int32, H_PRIME=torch.float32, STATUS=torch.int32, PASS_BITS=torch.int64)


def _check(code: int, what: str):
    if code != 0:
        raise HydraError("%s: %s (%d) %s" % (what, lib.hydra_status_str(code).decode(), code,
                                             lib.hydra_last_error().decode()))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _ptr_array(tensors: Sequence[Optional[torch.Tensor]]):
    arr = (C.c_void_p * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        arr[i] = _ptr(t)
    return arr


class Hydra:
    """One decoding context (hydra_create .. hydra_destroy).  `weights` maps the names of synth.weights
    (embed, lm_head, final_norm, L{l}.*, P.*, H{i}.*) to CUDA tensors, row-major [out][in]."""

    def __init__(self, model, head, parent: Sequence[int], weights: Dict[str, torch.Tensor], max_batch: int, max_seq: int):
        self.model, self.head, self.parent = model, head, list(parent)
        self.T = len(parent)
        self.K = head.n_heads
        self.max_batch, self.max_seq = max_batch, max_seq
        self.dtype = torch.float32 if model.dtype == "fp32" else torch.bfloat16
        self._w = weights                                   # keep the tensors alive
        for name, t in weights.items():
            if not t.is_cuda or not t.is_contiguous() or t.dtype != self.dtype:
                raise HydraError("weight %s must be a contiguous CUDA tensor of %s" % (name, self.dtype))
        self._mc = ModelCfgC(model.n_layers, model.d_model, model.n_heads, model.head_dim, model.d_ffn, model.vocab,
                             model.rms_eps, model.rope_theta, 0 if model.dtype == "fp32" else 1, max_batch, max_seq,
                             int(getattr(model, "kv_planes", 2)))
        self.kv_planes = 1 if model.dtype == "fp32" else (1 if self._mc.kv_planes == 1 else 2)
        self._hc = HeadCfgC(head.n_heads, head.n_mlp_layers, int(head.prefix_attn), int(head.has_bias),
                            int(getattr(head, "medusa", False)))
        self._parent_arr = (C.c_int32 * self.T)(*self.parent)
        self._tc = TreeCfgC(self.T, self._parent_arr)
        nbytes = lib.hydra_workspace_bytes(C.byref(self._mc), C.byref(self._hc), C.byref(self._tc))
        if nbytes == 0:
            raise HydraError("invalid configuration")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        self._ws_off = (-self.workspace.data_ptr()) % 256
        L = range(model.n_layers)
        g = weights.get
        self._arrs = [_ptr_array([g("L%d.%s" % (l, n)) for l in L])
                      for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")]
        self._arrs += [_ptr_array([g("H%d.%s" % (i, n)) for i in range(1, head.n_heads + 1)])
                       for n in ("w1", "b1", "wr", "br")]
        wc = WeightsC(_ptr(g("embed")), _ptr(g("lm_head")), _ptr(g("final_norm")),
                      *[C.cast(a, _PP) for a in self._arrs],
                      *[_ptr(g("P." + n)) for n in ("attn_norm", "wqkv", "wo", "ffn_norm", "w_gate_up", "w_down")])
        self._ctx = C.c_void_p()
        _check(lib.hydra_create(C.byref(self._ctx), C.byref(self._mc), C.byref(self._hc), C.byref(self._tc), C.byref(wc),
                                self.workspace.data_ptr() + self._ws_off, nbytes), "hydra_create")
        self.batch = 0

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            lib.hydra_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the calls of the C ABI
    def prefill(self, prompts: List[torch.Tensor]):
        self.batch = len(prompts)
        offs = [0]
        for p in prompts:
            offs.append(offs[-1] + p.numel())
        toks = torch.cat([p.to(torch.int32).flatten() for p in prompts]).cuda()
        arr = (C.c_int32 * len(offs))(*offs)
        _check(lib.hydra_prefill(self._ctx, self.batch, toks.data_ptr(), arr, _stream()), "hydra_prefill")
        torch.cuda.current_stream().synchronize()          # toks may be freed after this returns

    def draft(self) -> torch.Tensor:
        tok = torch.empty(self.batch, self.T, dtype=torch.int32, device="cuda")
        _check(lib.hydra_draft(self._ctx, tok.data_ptr(), _stream()), "hydra_draft")
        return tok

    def verify(self, tree_tok: torch.Tensor, want_logits: bool = False):
        assert tree_tok.dtype == torch.int32 and tree_tok.is_cuda and tree_tok.is_contiguous()
        amax = torch.empty(self.batch, self.T, dtype=torch.int32, device="cuda")
        logits = torch.empty(self.batch, self.T, self.model.vocab, dtype=torch.float32, device="cuda") if want_logits else None
        _check(lib.hydra_verify(self._ctx, tree_tok.data_ptr(), amax.data_ptr(), _ptr(logits), _stream()), "hydra_verify")
        return (amax, logits) if want_logits else amax

    def accept_compact(self, tree_tok: torch.Tensor, amax: torch.Tensor):
        n_acc = torch.empty(self.batch, dtype=torch.int32, device="cuda")
        path = torch.empty(self.batch, self.K + 1, dtype=torch.int32, device="cuda")
        out = torch.empty(self.batch, self.K + 1, dtype=torch.int32, device="cuda")
        _check(lib.hydra_accept_compact(self._ctx, tree_tok.data_ptr(), amax.data_ptr(), n_acc.data_ptr(), path.data_ptr(),
                                        out.data_ptr(), _stream()), "hydra_accept_compact")
        return n_acc, path, out

    def step(self, n_acc: Optional[torch.Tensor] = None, out_tok: Optional[torch.Tensor] = None):
        if n_acc is None:
            n_acc = torch.empty(self.batch, dtype=torch.int32, device="cuda")
        if out_tok is None:
            out_tok = torch.empty(self.batch, self.K + 1, dtype=torch.int32, device="cuda")
        _check(lib.hydra_step(self._ctx, n_acc.data_ptr(), out_tok.data_ptr(), _stream()), "hydra_step")
        return n_acc, out_tok

    def set_plant(self, plant: Optional[torch.Tensor]):
        self._plant = plant
        _check(lib.hydra_set_plant(self._ctx, _ptr(plant)), "hydra_set_plant")

    def set_acceptance(self, mode: int, tau: float = 1.0, eps: float = 0.0, alpha: float = 0.0,
                       u: Optional[torch.Tensor] = None):
        """hydra_set_acceptance: 0 greedy, 1 typical (tau, eps, alpha); u: float32 CUDA tensor [max_batch] of uniform
        numbers for the token after the accepted path, or None (its most likely token)."""
        if u is not None:
            _dense_cuda(u, torch.float32, "u")
            _need(u.numel() >= self.max_batch, "u [max_batch]")
        self._u = u
        _check(lib.hydra_set_acceptance(self._ctx, mode, tau, eps, alpha, _ptr(u)), "hydra_set_acceptance")

    def set_gemm_mode(self, mode: int):
        _check(lib.hydra_set_gemm_mode(self._ctx, mode), "hydra_set_gemm_mode")

    def set_step_graph(self, on: bool):
        _check(lib.hydra_set_step_graph(self._ctx, int(on)), "hydra_set_step_graph")

    def set_timing(self, on: bool):
        _check(lib.hydra_set_timing(self._ctx, int(on)), "hydra_set_timing")

    def get_timing(self, kclass: int):
        """(ms_total, launches, algorithmic_bytes) of a kernel class: 0 GEMM, 1 tree attention, 2 accept+compact."""
        ms, n, by = C.c_double(), C.c_longlong(), C.c_double()
        _check(lib.hydra_get_timing(self._ctx, kclass, C.byref(ms), C.byref(n), C.byref(by)), "hydra_get_timing")
        return ms.value, n.value, by.value

    def poll_status(self):
        _check(lib.hydra_poll_status(self._ctx, _stream()), "hydra_poll_status")

    def launch_count(self) -> int:
        return int(lib.hydra_launch_count(self._ctx))

    def get_buffer(self, name: str) -> torch.Tensor:
        """A tensor view of a library buffer (flat; KV buffers in the cache element type: float32 on the float path,
        float16 on the bfloat16 path)."""
        p, n = C.c_void_p(), C.c_size_t()
        _check(lib.hydra_get_buffer(self._ctx, BUF[name], C.byref(p), C.byref(n)), "hydra_get_buffer")
        off = p.value - self.workspace.data_ptr()
        cache_dtype = torch.float32 if self.dtype == torch.float32 else torch.float16
        return self.workspace[off:off + n.value].view(_BUF_DTYPE.get(name, cache_dtype))


# ---- single-kernel entry points (kernel-level parity tests)
def _need(cond: bool, what: str):
    if not cond:
        raise HydraError("bad argument: " + what)


def _dense_cuda(t: torch.Tensor, dtype, name: str):
    _need(isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype,
          "%s must be a contiguous CUDA tensor of %s" % (name, dtype))


def gemm(x: torch.Tensor, w: torch.Tensor, mode: int = 0) -> torch.Tensor:
    """out[m][n] = sum_k x[m][k] w[n][k] in float; x, w both float32 or both bfloat16 CUDA tensors.
    x may be [2][m][k] bfloat16: the hi = bf16(v) and lo = bf16(v - hi) planes of float activations v."""
    planes = 2 if x.dim() == 3 else 1
    m, k = x.shape[-2:]
    n = w.shape[0]
    _need(x.dtype in (torch.float32, torch.bfloat16), "x must be float32 or bfloat16")
    _dense_cuda(x, x.dtype, "x")
    _dense_cuda(w, x.dtype, "w")
    _need(w.dim() == 2 and w.shape[1] == k and (planes == 1 or x.shape[0] == 2), "x [m][k] or [2][m][k], w [n][k]")
    dtype = 0 if x.dtype == torch.float32 else 1
    out = torch.empty(m, n, dtype=torch.float32, device="cuda")
    part = torch.empty(lib.hydra_gemm_partial_floats(m, n, k, dtype, mode), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    _check(lib.hydra_gemm(x.data_ptr(), w.data_ptr(), out.data_ptr(), part.data_ptr(), m, n, k, dtype, mode, planes,
                          status.data_ptr(), _stream()), "hydra_gemm")
    word = int(status.item())
    if word:
        raise HydraError("hydra_gemm device status word %d" % word)
    return out


def gemm_noalloc(x: torch.Tensor, w: torch.Tensor, out: torch.Tensor, status: torch.Tensor):
    """hydra_gemm_noalloc: bfloat16 tensor-core GEMM whose partial sums live in the library's built-in 8 MiB scratch.
    The caller passes every tensor (nothing is allocated here, on the host side either): x [m][k], w [n][k]
    bfloat16, out [m][n] float32, status int32[1].  Calls that overlap on the GPU race on the scratch."""
    _dense_cuda(x, torch.bfloat16, "x")
    _dense_cuda(w, torch.bfloat16, "w")
    _dense_cuda(out, torch.float32, "out")
    _dense_cuda(status, torch.int32, "status")
    _need(x.dim() == 2 and w.dim() == 2 and w.shape[1] == x.shape[1], "x [m][k], w [n][k]")
    m, k = x.shape
    n = w.shape[0]
    _need(tuple(out.shape) == (m, n) and status.numel() >= 1, "out [m][n], status int32[>=1]")
    _check(lib.hydra_gemm_noalloc(x.data_ptr(), w.data_ptr(), out.data_ptr(), m, n, k, status.data_ptr(), _stream()),
           "hydra_gemm_noalloc")


def tree_attention(q, k_cache, v_cache, pos0, n_rows, mask, tc: int, out_planes: int = 1) -> torch.Tensor:
    """hydra_tree_attention.  q [batch*tc][H][hd], caches [batch][H][S][hd]: all float32, or all float16 (the bfloat16
    model path, whose result is bfloat16 in out_planes planes: [rows][H*hd] or [2][rows][H*hd] = hi, lo).  float16 inputs
    may carry a leading axis of 2: the hi = f16(v) and lo = f16(v - hi) planes.
    mask: int64 [tc] ancestor bitmasks, or None for a causal chunk (float16 only)."""
    planes = 2 if k_cache.dim() == 5 else 1
    batch, n_heads, max_seq, head_dim = k_cache.shape[-4:]
    _need(k_cache.dtype in (torch.float32, torch.float16), "caches must be float32 or float16")
    for name, t in (("q", q), ("k_cache", k_cache), ("v_cache", v_cache)):
        _dense_cuda(t, k_cache.dtype, name)
    _need(v_cache.shape == k_cache.shape and q.numel() == planes * batch * tc * n_heads * head_dim, "q / cache shapes")
    _need(planes == 1 or k_cache.dtype == torch.float16, "two planes: float16 only")
    _dense_cuda(pos0, torch.int32, "pos0")
    _need(pos0.numel() == batch and (n_rows is None or n_rows.numel() == batch), "pos0 [batch], n_rows [batch]")
    if mask is not None:
        _dense_cuda(mask, torch.int64, "mask")
        _need(mask.numel() == tc, "mask [tc]")
    if n_rows is not None:
        _dense_cuda(n_rows, torch.int32, "n_rows")
    shape = (batch * tc, n_heads * head_dim)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if k_cache.dtype == torch.float32:
        _need(mask is not None and out_planes == 1, "the float path needs a mask and has one output plane")
        out = torch.empty(shape, dtype=torch.float32, device="cuda")
        scratch = torch.empty(lib.hydra_attention_scratch_bytes(batch, tc, n_heads, head_dim, max_seq), dtype=torch.uint8,
                              device="cuda")
        dtype = 0
    else:
        out = torch.empty((2,) + shape if out_planes == 2 else shape, dtype=torch.bfloat16, device="cuda")
        scratch, dtype = None, 1
    _check(lib.hydra_tree_attention(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), pos0.data_ptr(), _ptr(n_rows),
                                    _ptr(mask), out.data_ptr(), _ptr(scratch), batch, tc, n_heads, head_dim,
                                    max_seq, dtype, planes, out_planes, status.data_ptr(), _stream()), "hydra_tree_attention")
    word = int(status.item())
    if word:
        raise HydraError("hydra_tree_attention device status word %d" % word)
    return out


def gemm_bounded_wait_probe(x: torch.Tensor, w: torch.Tensor, skip_unit: int, wait_limit: int = 1024,
                            status_words: Optional[torch.Tensor] = None):
    """hydra_gemm_bounded_wait_probe: a one-CTA tensor-core GEMM whose weight tile `skip_unit` is never requested,
    so a bounded wait runs out.  Returns (status word, diag int32[8]) as CPU values.  status_words: an int32[>=16]
    CUDA tensor to use as status word ([0]) and diagnostics ([8..15]), e.g. a context's STATUS buffer."""
    _dense_cuda(x, torch.bfloat16, "x")
    _dense_cuda(w, torch.bfloat16, "w")
    m, k = x.shape
    n = w.shape[0]
    _need(w.shape[1] == k, "w [n][k]")
    part = torch.empty(lib.hydra_gemm_partial_floats(m, n, k, 1, 0), dtype=torch.float32, device="cuda")
    if status_words is None:
        status_words = torch.zeros(16, dtype=torch.int32, device="cuda")
    _dense_cuda(status_words, torch.int32, "status_words")
    _need(status_words.numel() >= 16, "status_words int32[>=16]")
    status, diag = status_words[0:1], status_words[8:16]
    _check(lib.hydra_gemm_bounded_wait_probe(x.data_ptr(), w.data_ptr(), part.data_ptr(), m, n, k, skip_unit, wait_limit,
                                             status.data_ptr(), diag.data_ptr(), _stream()), "hydra_gemm_bounded_wait_probe")
    torch.cuda.current_stream().synchronize()
    return int(status.item()), diag.cpu().tolist()
