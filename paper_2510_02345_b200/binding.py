"""Thin ctypes binding over libcmoe.so: argument marshalling only.

The functions carry the names of the C boundary (include/cmoe.h).  PyTorch is
used for device memory and streams; every step of the layer runs in the
library's CUDA kernels.  There is no CPU fallback: if the shared library is
missing or no CUDA device is present, loading or calling fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG, "libcmoe.so")

CMOE_OK = 0
ERRORS = {
    -1: "CMOE_ERR_INVALID_ARG", -2: "CMOE_ERR_UNSUPPORTED_SHAPE", -3: "CMOE_ERR_WORKSPACE_TOO_SMALL",
    -4: "CMOE_ERR_T_EXCEEDS_MAX", -5: "CMOE_ERR_CUDA", -6: "CMOE_ERR_TIMEOUT",
}
EXPORTS = ["cmoe_compress_workspace_bytes", "cmoe_compress", "cmoe_quantize_int4", "cmoe_expert_similarity",
           "cmoe_workspace_bytes", "cmoe_workspace_bytes_ex", "cmoe_create", "cmoe_create_ex", "cmoe_selftest_wait_timeout", "cmoe_expert_stats", "cmoe_route", "cmoe_forward", "cmoe_forward_host", "cmoe_status",
           "cmoe_get_info", "cmoe_last_cuda_error", "cmoe_destroy", "cmoe_strerror",
           "cmoe_profile_enable", "cmoe_profile_read", "cmoe_stage_name", "cmoe_route_static"]
CMOE_MAX_STAGES = 8


class CmoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {ERRORS.get(code, code)} ({strerror(code)})")


class cmoe_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("d", "d_ff", "E", "G", "r", "k", "quant_group", "T_max")] + [
        (n, C.c_void_p) for n in ("C", "R", "b_c", "b_e", "B1", "B2", "U1q", "V1q", "U2q", "V2q",
                                  "U1s", "V1s", "U2s", "V2s", "expert_global_id", "workspace")
    ] + [("workspace_bytes", C.c_size_t)]


class cmoe_options(C.Structure):
    _fields_ = [("force_path", C.c_int32), ("router_fp32", C.c_int32), ("up_tile", C.c_int32), ("base_dtype", C.c_int32),
                ("host_chunks", C.c_int32), ("row_gather", C.c_int32), ("clusters_per_token", C.c_int32), ("move_in_scatter", C.c_int32)]


class cmoe_compress_desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("d_in", "d_out", "E", "G", "r", "oversample", "power_iters")] + [("gamma", C.c_float)] + [
        (n, C.c_void_p) for n in ("W", "omega", "B", "Uq", "Us", "Vq", "Vs", "sigma", "rel_err", "cosine", "pruned",
                                  "A_out", "Bt_out", "workspace")] + [("workspace_bytes", C.c_size_t)]


class cmoe_similarity_desc(C.Structure):
    _fields_ = [("E", C.c_int32), ("d", C.c_int32), ("n", C.c_int64), ("alpha", C.c_float)] + [
        (n, C.c_void_p) for n in ("W", "mu", "S_param", "S_task", "S", "status")]


class cmoe_info(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("path", "launches_route", "launches_forward", "row_align", "T_pad_max",
                                         "memsets_forward", "n_stages", "pruned_blocks")]


_lib = None


def lib():
    """Load libcmoe.so (built in-tree by paper_2510_02345_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2510_02345_b200.build` "
                "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        L.cmoe_workspace_bytes.argtypes = [C.POINTER(cmoe_desc), C.POINTER(C.c_size_t)]
        L.cmoe_create.argtypes = [C.POINTER(cmoe_desc), C.POINTER(C.c_void_p)]
        L.cmoe_workspace_bytes_ex.argtypes = [C.POINTER(cmoe_desc), C.POINTER(cmoe_options), C.POINTER(C.c_size_t)]
        L.cmoe_compress_workspace_bytes.argtypes = [C.POINTER(cmoe_compress_desc), C.POINTER(C.c_size_t)]
        L.cmoe_compress.argtypes = [C.POINTER(cmoe_compress_desc), C.c_void_p]
        L.cmoe_quantize_int4.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.cmoe_expert_similarity.argtypes = [C.POINTER(cmoe_similarity_desc), C.c_void_p]
        L.cmoe_create_ex.argtypes = [C.POINTER(cmoe_desc), C.POINTER(cmoe_options), C.POINTER(C.c_void_p)]
        L.cmoe_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.cmoe_expert_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                        C.c_void_p, C.c_void_p]
        L.cmoe_route.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.cmoe_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.cmoe_forward_host.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.cmoe_status.argtypes = [C.c_void_p, C.c_void_p]
        L.cmoe_get_info.argtypes = [C.c_void_p, C.POINTER(cmoe_info)]
        L.cmoe_last_cuda_error.argtypes = [C.c_void_p]
        L.cmoe_destroy.argtypes = [C.c_void_p]
        L.cmoe_strerror.argtypes = [C.c_int]
        L.cmoe_strerror.restype = C.c_char_p
        L.cmoe_profile_enable.argtypes = [C.c_void_p, C.c_int]
        L.cmoe_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.cmoe_stage_name.argtypes = [C.c_void_p, C.c_int32]
        L.cmoe_stage_name.restype = C.c_char_p
        L.cmoe_route_static.argtypes = [C.c_int32] * 4 + [C.c_void_p] * 5 + [C.c_int32] + [C.c_void_p] * 4
        for name in EXPORTS:
            if name not in ("cmoe_strerror", "cmoe_stage_name"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().cmoe_strerror(code).decode()


def _check(rc: int, where: str):
    if rc != CMOE_OK:
        raise CmoeError(rc, where)


# ---- the C calls, one Python function each ------------------------------------------------------
def cmoe_workspace_bytes(desc: cmoe_desc) -> int:
    out = C.c_size_t(0)
    _check(lib().cmoe_workspace_bytes(C.byref(desc), C.byref(out)), "cmoe_workspace_bytes")
    return out.value


def cmoe_create(desc: cmoe_desc) -> C.c_void_p:
    handle = C.c_void_p()
    _check(lib().cmoe_create(C.byref(desc), C.byref(handle)), "cmoe_create")
    return handle


def cmoe_create_ex(desc: cmoe_desc, options: "cmoe_options | None") -> C.c_void_p:
    handle = C.c_void_p()
    _check(lib().cmoe_create_ex(C.byref(desc), C.byref(options) if options is not None else None, C.byref(handle)),
           "cmoe_create_ex")
    return handle


def cmoe_selftest_wait_timeout(handle, limit_cycles: int, stream: int):
    _check(lib().cmoe_selftest_wait_timeout(handle, limit_cycles, stream), "cmoe_selftest_wait_timeout")


def cmoe_expert_stats(handle, x_ptr: int, T: int, loads_ptr: int, xbar_ptr, mu_ptr, beta: float, cov_ptr, stream: int):
    _check(lib().cmoe_expert_stats(handle, x_ptr, T, loads_ptr, xbar_ptr, mu_ptr, beta, cov_ptr, stream), "cmoe_expert_stats")


def cmoe_route(handle, x_ptr: int, T: int, cluster_id_ptr: int, expert_ids_ptr: int, gates_ptr: int, stream: int):
    _check(lib().cmoe_route(handle, x_ptr, T, cluster_id_ptr, expert_ids_ptr, gates_ptr, stream), "cmoe_route")


def cmoe_forward(handle, x_ptr: int, T: int, y_ptr: int, stream: int):
    _check(lib().cmoe_forward(handle, x_ptr, T, y_ptr, stream), "cmoe_forward")


def cmoe_forward_host(handle, x_host_ptr: int, T: int, y_host_ptr: int, x_stage_ptr: int, y_stage_ptr: int, stream: int):
    _check(lib().cmoe_forward_host(handle, x_host_ptr, T, y_host_ptr, x_stage_ptr, y_stage_ptr, stream), "cmoe_forward_host")


def cmoe_status(handle, stream: int) -> int:
    return lib().cmoe_status(handle, stream)


def cmoe_get_info(handle) -> cmoe_info:
    info = cmoe_info()
    _check(lib().cmoe_get_info(handle, C.byref(info)), "cmoe_get_info")
    return info


def cmoe_profile_enable(handle, on: bool):
    _check(lib().cmoe_profile_enable(handle, 1 if on else 0), "cmoe_profile_enable")


def cmoe_profile_read(handle) -> dict:
    """{stage name: milliseconds} of the last profiled cmoe_forward on this handle."""
    ms = (C.c_float * CMOE_MAX_STAGES)()
    n = C.c_int32(0)
    _check(lib().cmoe_profile_read(handle, ms, C.byref(n)), "cmoe_profile_read")
    return {lib().cmoe_stage_name(handle, i).decode(): float(ms[i]) for i in range(n.value)}


def cmoe_route_static(d: int, E: int, G: int, k: int, C_ptr, R_ptr, b_c_ptr, b_e_ptr, x_ptr, T: int,
                      cluster_id_ptr, expert_ids_ptr, gates_ptr, stream: int):
    """Handle-free routing for callers that cannot allocate: the library's fixed device array is
    the only scratch (see include/cmoe.h).  Raises CmoeError on a non-zero return code."""
    _check(lib().cmoe_route_static(d, E, G, k, C_ptr, R_ptr, b_c_ptr, b_e_ptr, x_ptr, T,
                                   cluster_id_ptr, expert_ids_ptr, gates_ptr, stream), "cmoe_route_static")


def cmoe_destroy(handle):
    _check(lib().cmoe_destroy(handle), "cmoe_destroy")


def compress(W, G: int, r: int, omega, gamma: float = 0.0, power_iters: int = 2):
    """cmoe_compress on CUDA tensors: W [E][d_in][d_out] fp32, omega [E][d_out][l] fp32 (l = r + oversample).
    Returns a dict of CUDA tensors: B (fp16), Uq, Us, Vq, Vs, sigma, rel_err, cosine, pruned, A, Bt."""
    import torch
    E, d_in, d_out = W.shape
    l = omega.shape[2]
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
    assert omega.is_cuda and omega.dtype == torch.float32 and omega.is_contiguous() and tuple(omega.shape) == (E, d_out, l)
    dev = W.device
    out = dict(B=torch.empty((G, d_in, d_out), dtype=torch.float16, device=dev),
               Uq=torch.empty((E, r * d_in // 2), dtype=torch.uint8, device=dev),
               Us=torch.empty((E, r * d_in // 32), dtype=torch.float16, device=dev),
               Vq=torch.empty((E, d_out * r // 2), dtype=torch.uint8, device=dev),
               Vs=torch.empty((E, d_out * r // 32), dtype=torch.float16, device=dev),
               sigma=torch.empty((E, r), dtype=torch.float32, device=dev),
               rel_err=torch.empty(E, dtype=torch.float32, device=dev),
               cosine=torch.empty(E, dtype=torch.float32, device=dev),
               pruned=torch.empty(E, dtype=torch.int32, device=dev),
               A=torch.empty((E, d_in, r), dtype=torch.float32, device=dev),
               Bt=torch.empty((E, r, d_out), dtype=torch.float32, device=dev))
    d = cmoe_compress_desc()
    d.d_in, d.d_out, d.E, d.G, d.r, d.oversample, d.power_iters, d.gamma = d_in, d_out, E, G, r, l - r, power_iters, gamma
    d.W, d.omega = W.data_ptr(), omega.data_ptr()
    for name, field in (("B", "B"), ("Uq", "Uq"), ("Us", "Us"), ("Vq", "Vq"), ("Vs", "Vs"), ("sigma", "sigma"),
                        ("rel_err", "rel_err"), ("cosine", "cosine"), ("pruned", "pruned"), ("A", "A_out"), ("Bt", "Bt_out")):
        setattr(d, field, out[name].data_ptr())
    need = C.c_size_t(0)
    _check(lib().cmoe_compress_workspace_bytes(C.byref(d), C.byref(need)), "cmoe_compress_workspace_bytes")
    ws = torch.empty(need.value + 256, dtype=torch.uint8, device=dev)
    d.workspace = (ws.data_ptr() + 255) // 256 * 256
    d.workspace_bytes = need.value
    _check(lib().cmoe_compress(C.byref(d), torch.cuda.current_stream(dev).cuda_stream), "cmoe_compress")
    out["_workspace"] = ws          # keeps the scratch alive until the caller has synchronised
    return out


def quantize_int4(w):
    """cmoe_quantize_int4 on a CUDA fp32 tensor (size a multiple of 32) -> (packed uint8, fp16 scales)."""
    import torch
    assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous() and w.numel() % 32 == 0
    q = torch.empty(w.numel() // 2, dtype=torch.uint8, device=w.device)
    s = torch.empty(w.numel() // 32, dtype=torch.float16, device=w.device)
    _check(lib().cmoe_quantize_int4(w.data_ptr(), w.numel(), q.data_ptr(), s.data_ptr(),
                                    torch.cuda.current_stream(w.device).cuda_stream), "cmoe_quantize_int4")
    return q, s


def expert_similarity(W=None, mu=None, alpha: float = 0.7, out: dict | None = None):
    """cmoe_expert_similarity on CUDA fp32 tensors: W [E][...] (flattened per expert) and / or mu [E][d].
    Returns a dict of CUDA tensors [E][E]: S_param (if W), S_task (if mu), S (if both), and the int32 status word;
    `out` = the dict of an earlier call with the same arguments' shapes, to write into its tensors again."""
    import torch
    ref = W if W is not None else mu
    E, dev = ref.shape[0], ref.device
    q = cmoe_similarity_desc()
    q.E, q.alpha = E, alpha
    if out is None:
        out = {"status": torch.zeros(1, dtype=torch.int32, device=dev)}
        for name, need in (("S_param", W is not None), ("S_task", mu is not None), ("S", W is not None and mu is not None)):
            if need:
                out[name] = torch.empty((E, E), dtype=torch.float32, device=dev)
    q.status = out["status"].data_ptr()
    if W is not None:
        assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous()
        q.W, q.n = W.data_ptr(), W[0].numel()
        q.S_param = out["S_param"].data_ptr()
    if mu is not None:
        assert mu.is_cuda and mu.dtype == torch.float32 and mu.is_contiguous() and mu.shape[0] == E
        q.mu, q.d = mu.data_ptr(), mu.shape[1]
        q.S_task = out["S_task"].data_ptr()
    if W is not None and mu is not None:
        q.S = out["S"].data_ptr()
    _check(lib().cmoe_expert_similarity(C.byref(q), torch.cuda.current_stream(dev).cuda_stream), "cmoe_expert_similarity")
    return out


# ---- convenience owner of the device buffers ---------------------------------------------------
class ClusteredMoELayer:
    """Uploads a layer (numpy arrays in the boundary layouts) and owns the arena.

    route(x) / forward(x) take CUDA fp16 tensors [T][d] and launch on torch's current stream.
    """

    _NP_FIELDS = (("C", np.float32), ("R", np.float32), ("b_c", np.float32), ("b_e", np.float32),
                  ("B1", np.float16), ("B2", np.float16),
                  ("U1q", np.uint8), ("V1q", np.uint8), ("U2q", np.uint8), ("V2q", np.uint8),
                  ("U1s", np.float16), ("V1s", np.float16), ("U2s", np.float16), ("V2s", np.float16),
                  ("expert_global_id", np.int32))

    def __init__(self, layer: dict, T_max: int | None = None, device: str = "cuda:0", keep_source: bool = False,
                 options: dict | None = None, guard_bytes: int = 0, fill_byte: int | None = None):
        """`options`: fields of cmoe_options (force_path, router_fp32, up_tile, clusters_per_token, ...) for cmoe_create_ex.
        `guard_bytes` / `fill_byte` (tests): the arena is allocated with that many bytes of a canary pattern
        before and after it, and filled with `fill_byte` before the library sees it."""
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU path)")
        s = layer["shape"]
        self.shape = s
        if layer.get("base_dtype", "fp16") == "bf16":         # B1, B2 are uint16 arrays of bfloat16 bits
            options = dict(options or {}, base_dtype=1)
        self.device = torch.device(device)
        self.T_max = int(T_max if T_max is not None else layer.get("T", s.T))
        torch.cuda.set_device(self.device)
        src = {}
        for name, dt in self._NP_FIELDS:
            a = layer.get(name)
            if a is None or a.size == 0:
                src[name] = None
            elif name in ("B1", "B2") and a.dtype == np.uint16:
                src[name] = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(self.device)   # bit patterns
            else:
                src[name] = torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(self.device)
        desc = cmoe_desc()
        desc.d, desc.d_ff, desc.E, desc.G, desc.r, desc.k = s.d, s.d_ff, s.E, s.G, s.r, s.k
        desc.quant_group, desc.T_max = 32, self.T_max
        for name, _ in self._NP_FIELDS:
            setattr(desc, name, None if src[name] is None else src[name].data_ptr())
        opts = None
        if options:
            opts = cmoe_options()
            opts.force_path = -1
            for key, val in options.items():
                setattr(opts, key, int(val))
        self.g1 = max(1, int(opts.clusters_per_token)) if opts is not None else 1
        need = C.c_size_t(0)
        _check(lib().cmoe_workspace_bytes_ex(C.byref(desc), C.byref(opts) if opts is not None else None, C.byref(need)),
               "cmoe_workspace_bytes_ex")
        nbytes = need.value
        guard = (int(guard_bytes) + 255) // 256 * 256
        self.workspace = torch.empty(nbytes + 256 + 2 * guard, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256 + guard
        off = base - self.workspace.data_ptr()
        if fill_byte is not None:
            self.workspace[off:off + nbytes] = int(fill_byte)
        self._guards = None
        if guard:
            self._guards = (self.workspace[off - guard:off], self.workspace[off + nbytes:off + nbytes + guard])
            for gbuf in self._guards:
                gbuf.fill_(0xA5)
        desc.workspace, desc.workspace_bytes = base, nbytes
        self.workspace_bytes = nbytes
        torch.cuda.synchronize(self.device)
        if opts is not None:
            self.handle = cmoe_create_ex(desc, opts)
        else:
            self.handle = cmoe_create(desc)
        self.info = cmoe_get_info(self.handle)
        self._src = src if keep_source else None   # the library holds its own copies in the arena

    def _stream(self) -> int:
        import torch
        return torch.cuda.current_stream(self.device).cuda_stream

    def route(self, x):
        import torch
        T = x.shape[0]
        k = self.shape.k
        assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.shape[1] == self.shape.d
        if self.g1 > 1:           # clusters_per_token: [T][g1], [T][g1][k], [T][g1][k]
            cid = torch.empty((T, self.g1), dtype=torch.int32, device=x.device)
            eid = torch.empty((T, self.g1, k), dtype=torch.int32, device=x.device)
            gates = torch.empty((T, self.g1, k), dtype=torch.float32, device=x.device)
        else:
            cid = torch.empty(T, dtype=torch.int32, device=x.device)
            eid = torch.empty((T, k), dtype=torch.int32, device=x.device)
            gates = torch.empty((T, k), dtype=torch.float32, device=x.device)
        cmoe_route(self.handle, x.data_ptr(), T, cid.data_ptr(), eid.data_ptr(), gates.data_ptr(), self._stream())
        return cid, eid, gates

    def forward(self, x, out=None):
        import torch
        T = x.shape[0]
        assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.shape[1] == self.shape.d
        y = out if out is not None else torch.empty_like(x)
        cmoe_forward(self.handle, x.data_ptr(), T, y.data_ptr(), self._stream())
        return y

    def forward_host(self, x_host, out_host=None):
        """Host tensors in and out (pinned memory lets the copies overlap the kernels); asynchronous on the
        current stream like forward().  The device staging buffers are kept by the module."""
        import torch
        T = x_host.shape[0]
        assert (not x_host.is_cuda) and x_host.dtype == torch.float16 and x_host.is_contiguous() and x_host.shape[1] == self.shape.d
        y = out_host if out_host is not None else torch.empty_like(x_host)
        if getattr(self, "_stage", None) is None or self._stage[0].shape[0] < T:
            self._stage = (torch.empty((max(T, 1), self.shape.d), dtype=torch.float16, device=self.device),
                           torch.empty((max(T, 1), self.shape.d), dtype=torch.float16, device=self.device))
        cmoe_forward_host(self.handle, x_host.data_ptr(), T, y.data_ptr(), self._stage[0].data_ptr(),
                          self._stage[1].data_ptr(), self._stream())
        return y

    def expert_stats(self, x, mu=None, beta: float = 0.05):
        """loads [E] int32, xbar [E][d] fp32, cov (0-d fp32) of routing x; `mu` ([E][d] fp32) is updated in place by Eq. 5."""
        import torch
        s = self.shape
        assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.shape[1] == s.d
        loads = torch.empty(s.E, dtype=torch.int32, device=x.device)
        xbar = torch.empty((s.E, s.d), dtype=torch.float32, device=x.device)
        cov = torch.empty((), dtype=torch.float32, device=x.device)
        if mu is not None:
            assert mu.is_cuda and mu.dtype == torch.float32 and mu.is_contiguous() and tuple(mu.shape) == (s.E, s.d)
        cmoe_expert_stats(self.handle, x.data_ptr(), x.shape[0], loads.data_ptr(), xbar.data_ptr(),
                          None if mu is None else mu.data_ptr(), beta, cov.data_ptr(), self._stream())
        return loads, xbar, cov

    def guards_intact(self) -> bool:
        """True if the canary bytes around the arena (guard_bytes) still hold their pattern."""
        return self._guards is None or all(bool((gbuf == 0xA5).all()) for gbuf in self._guards)

    def status(self) -> int:
        return cmoe_status(self.handle, self._stream())

    def close(self):
        if getattr(self, "handle", None):
            cmoe_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
