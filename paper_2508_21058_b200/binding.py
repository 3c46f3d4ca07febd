"""ctypes binding of ``libmoc.so``.  Same names as the C entry points (include/moc.h);
argument marshalling only.  torch supplies device memory and the stream."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_DIR = os.path.dirname(os.path.abspath(__file__))
FLAG_CAUSAL = 0x1
WHOLE_SHOT = -1


class MocError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(what)
        self.code = code


class _Problem(C.Structure):
    _fields_ = [("n_heads", C.c_int32), ("n_tokens", C.c_int32), ("head_dim", C.c_int32),
                ("n_chunks", C.c_int32), ("top_k", C.c_int32), ("win_back", C.c_int32), ("win_fwd", C.c_int32),
                ("flags", C.c_uint32), ("softmax_scale", C.c_float),
                ("chunk_off", C.c_void_p), ("chunk_shot", C.c_void_p), ("chunk_mod", C.c_void_p)]


_lib = None


def lib_path() -> str:
    """The library this process loads: libmoc.so beside this file, or (MOC_LIBRARY=debug) the build with
    index checks, libmoc_debug.so."""
    return os.path.join(_DIR, "libmoc_debug.so" if os.environ.get("MOC_LIBRARY") == "debug" else "libmoc.so")


def load_library():
    """dlopen the CUDA library.  Raises if it has not been built: nothing else can run the path."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise MocError(-100, f"{path} is missing: build it with `python -m paper_2508_21058_b200.build` "
                             "(there is no fallback implementation)")
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    lib.moc_plan_create.argtypes = [C.POINTER(_Problem), C.POINTER(vp)]
    lib.moc_plan_destroy.argtypes = [vp]
    lib.moc_workspace_bytes.argtypes = [vp, i32, C.POINTER(sz)]
    lib.moc_chunk_pool.argtypes = [vp, vp, vp, vp, vp]
    lib.moc_chunk_pool_noalloc.argtypes = [vp, vp, vp, vp]
    lib.moc_plan_set_workspace_budget.argtypes = [vp, sz]
    lib.moc_route.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.moc_lists_from_sel.argtypes = [vp, vp, vp, vp]
    lib.moc_outer_num_shots.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.moc_outer_route.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.c_int32, vp, vp, vp, vp, vp]
    lib.moc_outer_reduced_layout.argtypes = [vp, vp, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                             vp, vp, vp, vp]
    lib.moc_gather_tokens.argtypes = [vp, vp, vp, C.c_int32, vp, vp]
    lib.moc_context_drop.argtypes = [vp, vp, C.c_float, C.c_float, C.c_uint64, vp, vp]
    # test hooks (exported, not in the public header)
    lib.moc_debug_use_cuda_core_attention.argtypes = [vp, i32]
    lib.moc_debug_set_wait_limit_us.argtypes = [vp, C.c_uint]
    lib.moc_debug_wait_probe.argtypes = [vp, vp, i32, vp]
    lib.moc_attend.argtypes = [vp] * 9
    lib.moc_attend_bwd.argtypes = [vp] * 13
    lib.moc_selected_pairs.argtypes = [vp, vp, vp, C.POINTER(C.c_int64)]
    lib.moc_get_status.argtypes = [vp, vp, vp, C.POINTER(i32), C.POINTER(i32)]
    lib.moc_launch_count.restype = C.c_int64
    lib.moc_strerror.restype = C.c_char_p
    lib.moc_strerror.argtypes = [i32]
    lib.moc_last_cuda_error.restype = C.c_char_p
    _lib = lib
    return lib


def launch_count() -> int:
    return int(load_library().moc_launch_count())


def _check(code: int):
    if code != 0:
        lib = load_library()
        msg = lib.moc_strerror(code).decode()
        if code == -7:
            msg += ": " + lib.moc_last_cuda_error().decode()
        raise MocError(code, f"moc error {code}: {msg}")


def _ptr(t):
    return C.c_void_p(0) if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class MocPlan:
    """Owns a ``moc_plan``.  Methods mirror the C entry points and take torch CUDA tensors."""

    def __init__(self, n_heads, n_tokens, head_dim, chunk_off, chunk_shot, chunk_mod, top_k,
                 win_back=0, win_fwd=0, causal=True, scalar_attend=False, softmax_scale=0.0):
        self._lib = load_library()
        self._h = C.c_void_p(0)
        off = np.ascontiguousarray(chunk_off, np.int32)
        shot = np.ascontiguousarray(chunk_shot, np.int32)
        mod = np.ascontiguousarray(chunk_mod, np.uint8)
        flags = FLAG_CAUSAL if causal else 0
        pr = _Problem(int(n_heads), int(n_tokens), int(head_dim), len(shot), int(top_k), int(win_back), int(win_fwd),
                      flags, float(softmax_scale), off.ctypes.data, shot.ctypes.data, mod.ctypes.data)
        if len(off) != len(shot) + 1 or len(mod) != len(shot):
            raise MocError(-3, "moc error -3: chunk tables have inconsistent lengths")
        _check(self._lib.moc_plan_create(C.byref(pr), C.byref(self._h)))
        self.H, self.L, self.d, self.C, self.k = int(n_heads), int(n_tokens), int(head_dim), len(shot), int(top_k)
        if scalar_attend:       # test hook: the in-library CUDA-core cross-check of the attention kernels
            _check(self._lib.moc_debug_use_cuda_core_attention(self._h, 1))

    @classmethod
    def from_workload(cls, wl, n_heads=None, **kw):
        lay = wl.layout
        return cls(wl.n_heads if n_heads is None else n_heads, lay.n_tokens, wl.head_dim, lay.chunk_off,
                   lay.chunk_shot, lay.chunk_mod, wl.top_k, wl.win_back, wl.win_fwd, wl.causal, **kw)

    def close(self):
        if self._h:
            self._lib.moc_plan_destroy(self._h)
            self._h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self, with_bwd=False) -> int:
        n = C.c_size_t(0)
        _check(self._lib.moc_workspace_bytes(self._h, int(with_bwd), C.byref(n)))
        return int(n.value)

    def moc_plan_set_workspace_budget(self, max_bytes: int):
        _check(self._lib.moc_plan_set_workspace_budget(self._h, C.c_size_t(int(max_bytes))))

    def new_workspace(self, with_bwd=False, device="cuda") -> torch.Tensor:
        return torch.empty(self.workspace_bytes(with_bwd), dtype=torch.uint8, device=device)

    def moc_chunk_pool(self, K, desc, ws):
        _check(self._lib.moc_chunk_pool(self._h, _ptr(K), _ptr(desc), _ptr(ws), _stream()))

    def moc_chunk_pool_noalloc(self, K, desc):
        """Descriptors without a workspace: scratch is a fixed array inside the library (small
        problems only; raises MocError -9 beyond its size).  Calls sharing a GPU must not overlap."""
        _check(self._lib.moc_chunk_pool_noalloc(self._h, _ptr(K), _ptr(desc), _stream()))

    def moc_route(self, Q, desc, sel_idx, ws):
        _check(self._lib.moc_route(self._h, _ptr(Q), _ptr(desc), _ptr(sel_idx), _ptr(ws), _stream()))

    def moc_lists_from_sel(self, sel_idx, ws):
        _check(self._lib.moc_lists_from_sel(self._h, _ptr(sel_idx), _ptr(ws), _stream()))

    def moc_context_drop(self, sel_idx, p_max, lam, seed, ws):
        _check(self._lib.moc_context_drop(self._h, _ptr(sel_idx), float(p_max), float(lam), int(seed), _ptr(ws), _stream()))

    def moc_attend(self, Q, K, V, sel_idx, O, lse, ws):
        _check(self._lib.moc_attend(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(sel_idx), _ptr(O), _ptr(lse), _ptr(ws),
                                    _stream()))

    def moc_attend_bwd(self, Q, K, V, O, lse, dO, sel_idx, dQ, dK, dV, ws):
        _check(self._lib.moc_attend_bwd(self._h, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse), _ptr(dO),
                                        _ptr(sel_idx), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws), _stream()))

    def moc_selected_pairs(self, ws) -> int:
        n = C.c_int64(0)
        _check(self._lib.moc_selected_pairs(self._h, _ptr(ws), _stream(), C.byref(n)))
        return int(n.value)

    def moc_get_status(self, ws):
        st, det = C.c_int(0), C.c_int(0)
        _check(self._lib.moc_get_status(self._h, _ptr(ws), _stream(), C.byref(st), C.byref(det)))
        return int(st.value), int(det.value)

    def moc_outer_num_shots(self) -> int:
        n = C.c_int32(0)
        _check(self._lib.moc_outer_num_shots(self._h, C.byref(n)))
        return int(n.value)

    def moc_outer_route(self, Xq, desc, q_tok0, q_tok1, top_m, shot_desc, scores, sel_shot, ws):
        _check(self._lib.moc_outer_route(self._h, _ptr(Xq), _ptr(desc), int(q_tok0), int(q_tok1), int(top_m), _ptr(shot_desc),
                                         _ptr(scores), _ptr(sel_shot), _ptr(ws), _stream()))

    def moc_outer_reduced_layout(self, sel_shot, q_tok0, q_tok1):
        """Host only: (chunk_off, chunk_shot, chunk_mod, tok_map) of the reduced stream for one row of sel_shot."""
        sel = np.ascontiguousarray(sel_shot, np.int32).reshape(-1)
        off = np.zeros(self.C + 1, np.int32)
        shot = np.zeros(self.C, np.int32)
        mod = np.zeros(self.C, np.uint8)
        tok = np.zeros(self.L, np.int32)
        nc, nt = C.c_int32(0), C.c_int32(0)
        _check(self._lib.moc_outer_reduced_layout(self._h, sel.ctypes.data, len(sel), int(q_tok0), int(q_tok1), C.byref(nc),
                                                  C.byref(nt), off.ctypes.data, shot.ctypes.data, mod.ctypes.data, tok.ctypes.data))
        return off[:nc.value + 1].copy(), shot[:nc.value].copy(), mod[:nc.value].copy(), tok[:nt.value].copy()

    def moc_gather_tokens(self, X, tok_map, out):
        _check(self._lib.moc_gather_tokens(self._h, _ptr(X), _ptr(tok_map), int(tok_map.numel()), _ptr(out), _stream()))

    # test hooks
    def debug_set_wait_limit_us(self, us: int):
        _check(self._lib.moc_debug_set_wait_limit_us(self._h, int(us)))

    def debug_wait_probe(self, ws, code: int):
        _check(self._lib.moc_debug_wait_probe(self._h, _ptr(ws), int(code), _stream()))

    # convenience: allocate outputs and run the forward path
    def forward(self, Q, K, V, ws=None):
        dev = Q.device
        ws = self.new_workspace(False, dev) if ws is None else ws
        desc = torch.empty((self.H, self.C, self.d), dtype=torch.float32, device=dev)
        sel = torch.empty((self.H, self.L, self.k), dtype=torch.int32, device=dev)
        O = torch.empty_like(Q)
        lse = torch.empty((self.H, self.L), dtype=torch.float32, device=dev)
        self.moc_chunk_pool(K, desc, ws)
        self.moc_route(Q, desc, sel, ws)
        self.moc_attend(Q, K, V, sel, O, lse, ws)
        return desc, sel, O, lse, ws
