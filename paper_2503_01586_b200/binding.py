"""ctypes binding of libelitekv.so: same names as the C ABI, argument marshalling only.

torch supplies device memory (`tensor.data_ptr()`) and the current stream; every step of the
path runs in the library's CUDA kernels.  There is no CPU or PyTorch fallback: if the shared
library is missing or fails to load, importing this module's functions raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ELITEKV_LIB", os.path.join(_HERE, "libelitekv.so"))

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_SHAPE = -2
ERR_WORKSPACE_TOO_SMALL = -3
ERR_CUDA = -4
ERR_TIMEOUT = -5
ERR_BAD_PAGE = -6
ERR_BAD_POSITION = -7
ERR_STATIC_SCRATCH_EXCEEDED = -8
STATIC_SCRATCH_BYTES = 48 << 20


class ElitekvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class Params(C.Structure):
    _fields_ = [("n_h", C.c_int32), ("d_h", C.c_int32), ("r", C.c_int32), ("d_c", C.c_int32),
                ("elite_idx", C.c_void_p), ("rope_base", C.c_float), ("softmax_scale", C.c_float),
                ("pair_mode", C.c_int32), ("W_uk", C.c_void_p), ("W_uv", C.c_void_p),
                ("max_pos", C.c_int32), ("cos_sin", C.c_void_p), ("decode_kernel", C.c_int32),
                ("d", C.c_int32), ("W_ke", C.c_void_p), ("W_down", C.c_void_p),
                ("d_ck", C.c_int32)]


class CacheDesc(C.Structure):
    _fields_ = [("rope", C.c_void_p), ("latent", C.c_void_p), ("page_table", C.c_void_p),
                ("page_size", C.c_int32), ("max_pages_per_seq", C.c_int32),
                ("num_pages", C.c_int64), ("max_ctx", C.c_int64), ("n_seqs", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_2503_01586_b200.build` (needs nvcc, sm_100a)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        L.elitekv_layer_create.argtypes = [C.POINTER(Params), C.POINTER(vp)]
        L.elitekv_layer_destroy.argtypes = [vp]
        L.elitekv_append.argtypes = [vp, C.POINTER(CacheDesc), vp, vp, vp, vp, i64, vp]
        L.elitekv_project_append.argtypes = [vp, C.POINTER(CacheDesc), vp, vp, vp, i64, vp]
        L.elitekv_absorb_query.argtypes = [vp, vp, vp, i32, vp, vp, vp]
        L.elitekv_decode_workspace_size.argtypes = [vp, i32, C.POINTER(sz)]
        L.elitekv_decode.argtypes = [vp, C.POINTER(CacheDesc), vp, vp, vp, i32, vp, sz, vp, vp]
        L.elitekv_decode_step.argtypes = [vp, C.POINTER(CacheDesc), vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, sz, vp, vp]
        L.elitekv_attend_rows_workspace_size.argtypes = [vp, i32, i32, C.POINTER(sz)]
        L.elitekv_attend_rows.argtypes = [vp, C.POINTER(CacheDesc), vp, vp, vp, i32, i32, vp, sz, vp, vp]
        L.elitekv_ropelite_workspace_size.argtypes = [i32, i32, i32, C.POINTER(sz)]
        L.elitekv_ropelite_distances.argtypes = [vp, vp, i32, i32, i32, C.c_float, vp, vp, sz, vp, vp]
        L.elitekv_ropelite_search.argtypes = [vp, vp, i32, i32, i32, C.c_float, i32, vp, sz, vp, vp, vp]
        L.elitekv_decode_static.argtypes = [vp, C.POINTER(CacheDesc), vp, vp, vp, i32, vp, vp]
        L.elitekv_plan.argtypes = [vp, i32, i32, i32, vp, vp, vp]
        L.elitekv_plan_workers.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.elitekv_decode_plan_info.argtypes = [vp, C.POINTER(CacheDesc), i32, C.POINTER(i32 * 5)]
        L.elitekv_check_status.argtypes = [vp, vp]
        L.elitekv_last_status_detail.argtypes = [vp, C.POINTER(i32 * 3)]
        L.elitekv_selftest_bounded_wait.argtypes = [vp, C.c_uint32, vp]
        L.elitekv_mha_workspace_size.argtypes = [i32, i32, i32, C.POINTER(sz)]
        L.elitekv_mha_decode.argtypes = [vp, vp, vp, vp, i32, i32, i32, i64, C.c_float, vp, sz, vp, vp]
        L.elitekv_profile_enable.argtypes = [vp, i32]
        L.elitekv_profile_collect.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(i32)]
        L.elitekv_strerror.argtypes = [C.c_int]
        L.elitekv_strerror.restype = C.c_char_p
        for name in ("elitekv_layer_create", "elitekv_layer_destroy", "elitekv_append",
                     "elitekv_absorb_query", "elitekv_decode_workspace_size", "elitekv_decode",
                     "elitekv_plan", "elitekv_check_status", "elitekv_mha_workspace_size",
                     "elitekv_profile_enable", "elitekv_profile_collect", "elitekv_decode_static",
                     "elitekv_mha_decode", "elitekv_plan_workers", "elitekv_decode_plan_info",
                     "elitekv_last_status_detail", "elitekv_selftest_bounded_wait",
                     "elitekv_project_append", "elitekv_decode_step",
                     "elitekv_attend_rows_workspace_size", "elitekv_attend_rows",
                     "elitekv_ropelite_workspace_size", "elitekv_ropelite_distances", "elitekv_ropelite_search"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().elitekv_strerror(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise ElitekvError(code, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous()
    return t.data_ptr()


def _dev(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.is_cuda and t.dtype == dtype and t.is_contiguous(), (t.device, t.dtype)
    return t


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Layer:
    """Owns an `elitekv_layer*`.  elite_idx is an int32 CPU tensor [n_h][r]; W_uk, W_uv are
    bf16 CUDA tensors; cos_sin an optional fp32 CUDA tensor [max_pos][d_h/2][2]."""

    def __init__(self, n_h, d_h, r, d_c, elite_idx, W_uk, W_uv, max_pos, rope_base=10000.0,
                 softmax_scale=0.0, pair_mode=0, cos_sin=None, decode_kernel=0, W_ke=None, W_down=None,
                 d_ck=0):
        idx = elite_idx.to(torch.int32).contiguous().cpu()
        assert tuple(idx.shape) == (n_h, r)
        self.n_h, self.d_h, self.r, self.d_c = n_h, d_h, r, d_c
        # separated latents (d_ck > 0): a latent row is [c_k (d_ck) | c_v (d_c - d_ck)]
        self.d_ck = d_ck
        self.kw = d_ck if d_ck > 0 else d_c          # width of the absorbed query
        self._keep = (idx, cos_sin)
        p = Params(n_h, d_h, r, d_c, idx.data_ptr() if r > 0 else None, rope_base, softmax_scale,
                   pair_mode, _ptr(W_uk) if W_uk is not None and W_uk.numel() else None,
                   _ptr(_dev(W_uv, torch.bfloat16)), max_pos,
                   _ptr(_dev(cos_sin, torch.float32)) if cos_sin is not None else None,
                   decode_kernel,
                   W_down.shape[0] if W_down is not None else 0,
                   _ptr(_dev(W_ke, torch.bfloat16)) if W_ke is not None else None,
                   _ptr(_dev(W_down, torch.bfloat16)) if W_down is not None else None, d_ck)
        h = C.c_void_p()
        _check(lib().elitekv_layer_create(C.byref(p), C.byref(h)), "elitekv_layer_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            lib().elitekv_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_cache(rope: torch.Tensor, latent: torch.Tensor, *, n_seqs: int, max_ctx: int = 0,
               page_table: Optional[torch.Tensor] = None, page_size: int = 64) -> CacheDesc:
    """Describes caller-owned cache planes.  Keep the tensors alive while the descriptor is used."""
    _dev(rope, torch.bfloat16)
    _dev(latent, torch.bfloat16)
    d = CacheDesc()
    d.rope, d.latent = rope.data_ptr(), latent.data_ptr()
    d.n_seqs = n_seqs
    if page_table is not None:
        _dev(page_table, torch.int32)
        d.page_table = page_table.data_ptr()
        d.page_size = page_size
        d.max_pages_per_seq = page_table.shape[1]
        d.num_pages = latent.shape[0] // page_size if latent.dim() == 2 else latent.shape[0]
        d.max_ctx = 0
    else:
        d.page_table = None
        d.page_size = page_size
        d.max_ctx = max_ctx
    return d


def elitekv_append(layer: Layer, cache: CacheDesc, k_e, c, seq_id, pos) -> None:
    T = c.shape[0]
    _check(lib().elitekv_append(layer.handle, C.byref(cache), _ptr(k_e), _ptr(_dev(c, torch.bfloat16)),
                                _ptr(_dev(seq_id, torch.int32)), _ptr(_dev(pos, torch.int32)), T,
                                _stream()), "elitekv_append")


def elitekv_project_append(layer: Layer, cache: CacheDesc, x, seq_id, pos) -> None:
    T = x.shape[0]
    _check(lib().elitekv_project_append(layer.handle, C.byref(cache), _ptr(_dev(x, torch.bfloat16)),
                                        _ptr(_dev(seq_id, torch.int32)), _ptr(_dev(pos, torch.int32)), T,
                                        _stream()), "elitekv_project_append")


def elitekv_absorb_query(layer: Layer, q, q_pos, q_rope=None, q_abs=None):
    B = q.shape[0]
    _dev(q, torch.bfloat16)
    if q_rope is None:
        q_rope = torch.empty((B, layer.n_h, 2 * layer.r), dtype=torch.bfloat16, device=q.device)
    if q_abs is None:
        q_abs = torch.empty((B, layer.n_h, layer.kw), dtype=torch.bfloat16, device=q.device)
    _check(lib().elitekv_absorb_query(layer.handle, _ptr(q), _ptr(_dev(q_pos, torch.int32)), B,
                                      _ptr(q_rope), _ptr(q_abs), _stream()), "elitekv_absorb_query")
    return q_rope, q_abs


def elitekv_decode_workspace_size(layer: Layer, B: int) -> int:
    n = C.c_size_t()
    _check(lib().elitekv_decode_workspace_size(layer.handle, B, C.byref(n)),
           "elitekv_decode_workspace_size")
    return n.value


def elitekv_decode(layer: Layer, cache: CacheDesc, q_rope, q_abs, seq_lens, workspace, out=None):
    B = q_abs.shape[0]
    if out is None:
        out = torch.empty((B, layer.n_h, layer.d_h), dtype=torch.bfloat16, device=q_abs.device)
    _check(lib().elitekv_decode(layer.handle, C.byref(cache), _ptr(q_rope), _ptr(_dev(q_abs, torch.bfloat16)),
                                _ptr(_dev(seq_lens, torch.int32)), B, workspace.data_ptr(),
                                workspace.numel() * workspace.element_size(), _ptr(out), _stream()),
           "elitekv_decode")
    return out


def elitekv_decode_step(layer: Layer, cache: CacheDesc, k_e, c, seq_id, pos, q, seq_lens, q_rope, q_abs,
                        workspace, out):
    """Append + query preparation + decode attention of one step in one call (buffers are the
    caller's: nothing is allocated here)."""
    B = q.shape[0]
    _check(lib().elitekv_decode_step(layer.handle, C.byref(cache), _ptr(k_e), _ptr(_dev(c, torch.bfloat16)),
                                     _ptr(_dev(seq_id, torch.int32)), _ptr(_dev(pos, torch.int32)),
                                     _ptr(_dev(q, torch.bfloat16)), _ptr(_dev(seq_lens, torch.int32)), B,
                                     _ptr(q_rope), _ptr(_dev(q_abs, torch.bfloat16)), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(),
                                     _ptr(_dev(out, torch.bfloat16)), _stream()), "elitekv_decode_step")
    return out


def elitekv_attend_rows_workspace_size(layer: Layer, B: int, m: int) -> int:
    n = C.c_size_t()
    _check(lib().elitekv_attend_rows_workspace_size(layer.handle, B, m, C.byref(n)),
           "elitekv_attend_rows_workspace_size")
    return n.value


def elitekv_attend_rows(layer: Layer, cache: CacheDesc, q_rope, q_abs, seq_lens, m: int, workspace, out=None):
    """q_rope [B][m][n_h][2r], q_abs [B][m][n_h][kw] -> out [B][m][n_h][d_h] (causal over the cache)."""
    B = seq_lens.shape[0]
    if out is None:
        out = torch.empty((B, m, layer.n_h, layer.d_h), dtype=torch.bfloat16, device=q_abs.device)
    _check(lib().elitekv_attend_rows(layer.handle, C.byref(cache), _ptr(q_rope), _ptr(_dev(q_abs, torch.bfloat16)),
                                     _ptr(_dev(seq_lens, torch.int32)), B, m, workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _ptr(out), _stream()),
           "elitekv_attend_rows")
    return out


def elitekv_ropelite_workspace_size(n_heads: int, n: int, d_h: int) -> int:
    b = C.c_size_t()
    _check(lib().elitekv_ropelite_workspace_size(n_heads, n, d_h, C.byref(b)), "elitekv_ropelite_workspace_size")
    return b.value


def _ropelite_ws(Q):
    H, n, d_h = Q.shape
    return torch.empty(elitekv_ropelite_workspace_size(H, n, d_h), dtype=torch.uint8, device=Q.device)


def elitekv_ropelite_distances(Q, K, rope_base: float = 10000.0, elite_mask=None, workspace=None):
    """Q, K bf16 [n_heads][n][d_h]; elite_mask optional int64 [n_heads] (bit i = chunk i chosen).
    Returns fp32 [n_heads][d_h/2]."""
    H, n, d_h = Q.shape
    ws = _ropelite_ws(Q) if workspace is None else workspace
    dist = torch.empty((H, d_h // 2), dtype=torch.float32, device=Q.device)
    _check(lib().elitekv_ropelite_distances(_ptr(_dev(Q, torch.bfloat16)), _ptr(_dev(K, torch.bfloat16)), H, n, d_h,
                                            rope_base, _ptr(_dev(elite_mask, torch.int64)) if elite_mask is not None else None,
                                            ws.data_ptr(), ws.numel(), _ptr(dist), _stream()),
           "elitekv_ropelite_distances")
    return dist


def elitekv_ropelite_search(Q, K, r: int, rope_base: float = 10000.0, trace: bool = False, workspace=None):
    """r greedy rounds for every head.  Returns int32 [n_heads][r] (and fp32 [r][n_heads][d_h/2])."""
    H, n, d_h = Q.shape
    ws = _ropelite_ws(Q) if workspace is None else workspace
    idx = torch.empty((H, r), dtype=torch.int32, device=Q.device)
    tr = torch.empty((r, H, d_h // 2), dtype=torch.float32, device=Q.device) if trace else None
    _check(lib().elitekv_ropelite_search(_ptr(_dev(Q, torch.bfloat16)), _ptr(_dev(K, torch.bfloat16)), H, n, d_h,
                                         rope_base, r, ws.data_ptr(), ws.numel(), _ptr(idx), _ptr(tr), _stream()),
           "elitekv_ropelite_search")
    return (idx, tr) if trace else idx


class DecodeStepRunner:
    """Host-to-host decode step of one layer at a fixed batch size B.  The step's six input
    arrays live in ONE pinned staging buffer (`host[...]`: k_e [B][n_h][2r], c [B][d_c],
    q [B][n_h][d_h], seq_id / pos / lens [B] int32) that crosses in one copy; the result comes
    back into the pinned `out_host` [B][n_h][d_h].  With `graph=True` the copy in, the
    elitekv_decode_step call and the copy out are captured in a CUDA graph on the second `run()`
    and replayed from then on; otherwise `run()` enqueues the three eagerly.  Marshalling only: every byte of
    arithmetic happens in the library's kernels."""

    ORDER = ("k_e", "c", "q", "seq_id", "pos", "lens")

    def __init__(self, layer: Layer, cache: CacheDesc, B: int, device, graph: bool = True):
        self.layer, self.cache, self.B = layer, cache, B
        bf, i32 = torch.bfloat16, torch.int32
        shapes = {"k_e": ((B, layer.n_h, 2 * layer.r), bf), "c": ((B, layer.d_c), bf),
                  "q": ((B, layer.n_h, layer.d_h), bf), "seq_id": ((B,), i32), "pos": ((B,), i32),
                  "lens": ((B,), i32)}
        offs, at = {}, 0
        for k in self.ORDER:
            shape, dt = shapes[k]
            n = 1
            for e in shape:
                n *= e
            offs[k] = (at, n * torch.empty((), dtype=dt).element_size())
            at = (at + offs[k][1] + 255) & ~255
        self.pack_host = torch.zeros(max(at, 256), dtype=torch.uint8).pin_memory()
        self.pack_dev = torch.zeros(max(at, 256), dtype=torch.uint8, device=device)

        def views(buf):
            return {k: buf[offs[k][0]:offs[k][0] + offs[k][1]].view(shapes[k][1]).view(shapes[k][0])
                    for k in self.ORDER}
        self.host, self.dev = views(self.pack_host), views(self.pack_dev)
        self.q_rope = torch.empty((B, layer.n_h, 2 * layer.r), dtype=bf, device=device)
        self.q_abs = torch.empty((B, layer.n_h, layer.kw), dtype=bf, device=device)
        self.out = torch.empty((B, layer.n_h, layer.d_h), dtype=bf, device=device)
        self.out_host = torch.empty((B, layer.n_h, layer.d_h), dtype=bf).pin_memory()
        self.workspace = torch.empty(elitekv_decode_workspace_size(layer, B), dtype=torch.uint8, device=device)
        self.h2d_bytes = self.pack_host.numel()
        self.d2h_bytes = self.out_host.numel() * self.out_host.element_size()
        self.graph = None
        self._want_graph, self._warm = graph, False

    def _enqueue(self):
        d = self.dev
        self.pack_dev.copy_(self.pack_host, non_blocking=True)
        elitekv_decode_step(self.layer, self.cache, d["k_e"], d["c"], d["seq_id"], d["pos"], d["q"], d["lens"],
                            self.q_rope, self.q_abs, self.workspace, self.out)
        self.out_host.copy_(self.out, non_blocking=True)

    def run(self, wait: bool = True):
        """One step from `host[...]` to `out_host`; with `wait`, returns once the result is there.
        Nothing runs before the first call (the staging buffer is the caller's to fill first):
        that call goes eagerly, the second one captures the graph."""
        if self._want_graph and self.graph is None and self._warm:
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._enqueue()
            self.graph = g
        if self.graph is not None:
            self.graph.replay()
        else:
            self._enqueue()
            self._warm = True
        if wait:
            torch.cuda.current_stream().synchronize()
        return self.out_host


def elitekv_decode_static(layer: Layer, cache: CacheDesc, q_rope, q_abs, seq_lens, out):
    """elitekv_decode with the library's built-in scratch: no workspace argument and no
    allocation, so `out` must be passed in (this wrapper allocates nothing either)."""
    B = q_abs.shape[0]
    _check(lib().elitekv_decode_static(layer.handle, C.byref(cache), _ptr(q_rope),
                                       _ptr(_dev(q_abs, torch.bfloat16)),
                                       _ptr(_dev(seq_lens, torch.int32)), B,
                                       _ptr(_dev(out, torch.bfloat16)), _stream()),
           "elitekv_decode_static")
    return out


def elitekv_plan(seq_lens, tile_tokens: int, max_items: int):
    B = seq_lens.shape[0]
    items = torch.empty((max_items, 4), dtype=torch.int32, device=seq_lens.device)
    first = torch.empty((B + 1,), dtype=torch.int32, device=seq_lens.device)
    _check(lib().elitekv_plan(_ptr(_dev(seq_lens, torch.int32)), B, tile_tokens, max_items,
                              _ptr(items), _ptr(first), _stream()), "elitekv_plan")
    return items, first


def elitekv_plan_workers(seq_lens, tile_tokens: int, n_workers: int, max_items: int,
                         item_overhead_tiles: int = 0):
    B = seq_lens.shape[0]
    items = torch.empty((max_items, 4), dtype=torch.int32, device=seq_lens.device)
    first = torch.empty((B + 1,), dtype=torch.int32, device=seq_lens.device)
    wfirst = torch.empty((n_workers + 1,), dtype=torch.int32, device=seq_lens.device)
    _check(lib().elitekv_plan_workers(_ptr(_dev(seq_lens, torch.int32)), B, tile_tokens, n_workers,
                                      item_overhead_tiles, max_items, _ptr(items), _ptr(first), _ptr(wfirst), _stream()),
           "elitekv_plan_workers")
    return items, first, wfirst


def elitekv_decode_plan_info(layer: Layer, cache: Optional[CacheDesc], B: int):
    """(kernel, tokens per plan tile, persistent workers, plan capacity, item overhead tiles)."""
    info = (C.c_int32 * 5)()
    _check(lib().elitekv_decode_plan_info(layer.handle, C.byref(cache) if cache is not None else None,
                                          B, C.byref(info)), "elitekv_decode_plan_info")
    return tuple(int(x) for x in info)


def elitekv_check_status(layer: Layer) -> int:
    return lib().elitekv_check_status(layer.handle, _stream())


def elitekv_last_status_detail(layer: Layer):
    """(detail0, detail1, fault count) read by the last elitekv_check_status of this layer."""
    d = (C.c_int32 * 3)()
    _check(lib().elitekv_last_status_detail(layer.handle, C.byref(d)), "elitekv_last_status_detail")
    return tuple(int(x) for x in d)


def elitekv_selftest_bounded_wait(layer: Layer, poll_limit: int) -> None:
    _check(lib().elitekv_selftest_bounded_wait(layer.handle, poll_limit, _stream()),
           "elitekv_selftest_bounded_wait")


def elitekv_profile_enable(layer: Layer, on: bool) -> None:
    _check(lib().elitekv_profile_enable(layer.handle, 1 if on else 0), "elitekv_profile_enable")


def elitekv_profile_collect(layer: Layer):
    """(summed split-K kernel milliseconds, launches) since the last collection."""
    ms, n = C.c_float(), C.c_int32()
    _check(lib().elitekv_profile_collect(layer.handle, C.byref(ms), C.byref(n)),
           "elitekv_profile_collect")
    return ms.value, n.value


def elitekv_mha_workspace_size(B: int, n_h: int, d_h: int) -> int:
    n = C.c_size_t()
    _check(lib().elitekv_mha_workspace_size(B, n_h, d_h, C.byref(n)), "elitekv_mha_workspace_size")
    return n.value


def elitekv_mha_decode(q_hat, K_hat, V, seq_lens, workspace, out=None, scale: float = 0.0):
    B, n_h, d_h = q_hat.shape
    max_ctx = K_hat.shape[1]
    if out is None:
        out = torch.empty_like(q_hat)
    _check(lib().elitekv_mha_decode(_ptr(_dev(q_hat, torch.bfloat16)), _ptr(_dev(K_hat, torch.bfloat16)),
                                    _ptr(_dev(V, torch.bfloat16)), _ptr(_dev(seq_lens, torch.int32)),
                                    B, n_h, d_h, max_ctx, scale, workspace.data_ptr(),
                                    workspace.numel() * workspace.element_size(), _ptr(out),
                                    _stream()), "elitekv_mha_decode")
    return out
