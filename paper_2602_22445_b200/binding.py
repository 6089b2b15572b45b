"""Thin ctypes binding of libftc.so: same names as the C ABI (include/ftc.h), argument marshalling only.

Device buffers are torch CUDA tensors (torch supplies memory and streams, nothing else); host buffers for
the *_host variants are numpy arrays or CPU tensors. There is no CPU or PyTorch fallback: if the library
is missing or fails to load, importing a function from here raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libftc.so")

FTC_I32, FTC_I64, FTC_U64, FTC_F32 = 0, 1, 2, 3
FTC_SUM, FTC_MAX, FTC_XOR = 0, 1, 2
FTC_OK, FTC_EINVAL, FTC_EUNSUPPORTED, FTC_EWORKSPACE, FTC_ECUDA, FTC_ETOOLARGE = 0, -1, -2, -3, -4, -5
FTC_NOALLOC_SCRATCH_BYTES = 8 << 20
FTC_ST_OK, FTC_ST_ROOT_FAILED, FTC_ST_NO_CLEAN_SUBTREE, FTC_ST_NO_LIVE_ROOT_CANDIDATE = 0, 1, 2, 3
FTC_ST_PRECONDITION_INOP_ROOT, FTC_ST_BAD_ROOT, FTC_ST_INTERNAL_TIMEOUT = 4, 5, 6
FTC_STATUS_WORDS = 4
FTC_MSG_WORDS = 8
FTC_INOP_UNUSED = 0xFFFFFFFF
FTC_OUT_EXPANDED = 0x1
FTC_KERNEL_GENERIC = 0x100
FTC_MAX_ARITY = 32
FTC_TREE_BINOMIAL = 0x1000000
FTC_PARTNERS_DESCENDING = 0x2000000


def FTC_TREE_ARITY(a: int) -> int:
    """Flag bits asking for a-ary heaps below the root's children."""
    return (a & 0xFF) << 16

FTC_KERNEL_DIRECT = 0x200
FTC_KERNEL_LEVELS = 0x400
FTC_DEBUG_ONE_POLL = 0x4000000
OPS = {"sum": FTC_SUM, "max": FTC_MAX, "xor": FTC_XOR}

EXPORTS = ["ftc_reduce_batch", "ftc_allreduce_batch", "ftc_reduce_batch_noalloc", "ftc_candidates_batch",
           "ftc_candidates_workspace_bytes", "ftc_candidates_kernel_name", "ftc_message_counts_batch", "ftc_failed_list_batch", "ftc_workspace_bytes", "ftc_reduce_batch_host",
           "ftc_allreduce_batch_host", "ftc_host_staging_bytes", "ftc_schedule_info", "ftc_fill_inputs",
           "ftc_kernel_name", "ftc_kernel_variant", "ftc_launch_blocks", "ftc_read_bandwidth_probe", "ftc_strerror", "ftc_version"]


class ftc_desc_t(C.Structure):
    _fields_ = [("P", C.c_uint32), ("f", C.c_uint32), ("k", C.c_uint32), ("dtype", C.c_uint32), ("op", C.c_uint32),
                ("root", C.c_int32), ("max_inop", C.c_uint32), ("flags", C.c_uint32)]


class ftc_sched_t(C.Structure):
    _fields_ = [("q", C.c_uint32), ("r", C.c_uint32), ("H", C.c_uint32), ("rounds_reduce", C.c_uint32),
                ("rounds_attempt", C.c_uint32), ("msgs_upcorrection", C.c_uint64), ("msgs_tree", C.c_uint64)]


class FtcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {ftc_strerror(code)} ({code})")


_lib = None


def load():
    """Load libftc.so (built in-tree by paper_2602_22445_b200.build). Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_22445_b200.build` "
                          "(there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, u64, u32, sz = C.c_void_p, C.c_uint64, C.c_uint32, C.c_size_t
    dp = C.POINTER(ftc_desc_t)
    batch_args = [dp, u64, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    for name in ("ftc_reduce_batch", "ftc_allreduce_batch", "ftc_reduce_batch_host", "ftc_allreduce_batch_host"):
        getattr(lib, name).restype = C.c_int
        getattr(lib, name).argtypes = batch_args
    lib.ftc_reduce_batch_noalloc.restype = C.c_int
    lib.ftc_reduce_batch_noalloc.argtypes = [dp, u64, vp, vp, vp, vp, vp, vp, vp]
    lib.ftc_candidates_batch.restype = C.c_int
    lib.ftc_candidates_batch.argtypes = [dp, u64, C.c_int, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.ftc_candidates_workspace_bytes.restype = sz
    lib.ftc_candidates_workspace_bytes.argtypes = [dp, u64]
    lib.ftc_candidates_kernel_name.restype = C.c_char_p
    lib.ftc_candidates_kernel_name.argtypes = [dp]
    lib.ftc_message_counts_batch.restype = C.c_int
    lib.ftc_message_counts_batch.argtypes = [dp, u64, C.c_int, vp, vp, vp, vp, vp]
    lib.ftc_failed_list_batch.restype = C.c_int
    lib.ftc_failed_list_batch.argtypes = [dp, u64, C.c_int, vp, vp, vp, vp, vp, vp]
    lib.ftc_workspace_bytes.restype = sz
    lib.ftc_workspace_bytes.argtypes = [dp, u64, C.c_int]
    lib.ftc_host_staging_bytes.restype = sz
    lib.ftc_host_staging_bytes.argtypes = [dp, u64]
    lib.ftc_schedule_info.restype = C.c_int
    lib.ftc_schedule_info.argtypes = [dp, C.POINTER(ftc_sched_t)]
    lib.ftc_fill_inputs.restype = C.c_int
    lib.ftc_fill_inputs.argtypes = [u32, u64, u64, u64, u32, u32, vp, vp]
    lib.ftc_kernel_name.restype = C.c_char_p
    lib.ftc_kernel_name.argtypes = [dp, C.c_int]
    lib.ftc_kernel_variant.restype = C.c_char_p
    lib.ftc_kernel_variant.argtypes = [dp, C.c_int]
    lib.ftc_launch_blocks.restype = C.c_int
    lib.ftc_launch_blocks.argtypes = [dp, u64, C.c_int, C.POINTER(u32)]
    lib.ftc_read_bandwidth_probe.restype = C.c_int
    lib.ftc_read_bandwidth_probe.argtypes = [u32, vp, u64, vp, vp]
    lib.ftc_strerror.restype = C.c_char_p
    lib.ftc_strerror.argtypes = [C.c_int]
    lib.ftc_version.restype = u32
    lib.ftc_version.argtypes = []
    _lib = lib
    return lib


def _torch():
    import torch
    return torch


def dtype_code(dt) -> int:
    """FTC_* code of a torch or numpy dtype."""
    name = str(dt).replace("torch.", "")
    return {"int32": FTC_I32, "int64": FTC_I64, "uint64": FTC_U64, "float32": FTC_F32}[name]


def make_desc(P, f, k, dtype, op, root=0, max_inop=0, flags=0) -> ftc_desc_t:
    return ftc_desc_t(P, f, k, dtype if isinstance(dtype, int) else dtype_code(dtype),
                      OPS[op] if isinstance(op, str) else op, root, max_inop, flags)


def _dev_ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device arguments must be contiguous CUDA tensors")
    return t.data_ptr()


def _host_ptr(a):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        if not a.flags["C_CONTIGUOUS"]:
            raise ValueError("host arrays must be C-contiguous")
        return a.ctypes.data
    if a.is_cuda or not a.is_contiguous():
        raise ValueError("host arguments must be contiguous CPU tensors or numpy arrays")
    return a.data_ptr()


def _stream(stream):
    if stream is None:
        return _torch().cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def ftc_strerror(code: int) -> str:
    return load().ftc_strerror(code).decode()


def ftc_version() -> int:
    return load().ftc_version()


def ftc_kernel_name(desc, is_allreduce=False) -> str:
    return load().ftc_kernel_name(C.byref(desc), int(is_allreduce)).decode()


def ftc_kernel_variant(desc, is_allreduce=False) -> str:
    return load().ftc_kernel_variant(C.byref(desc), int(is_allreduce)).decode()


def ftc_launch_blocks(desc, S, is_allreduce=False) -> int:
    out = C.c_uint32(0)
    rc = load().ftc_launch_blocks(C.byref(desc), S, int(is_allreduce), C.byref(out))
    if rc != FTC_OK:
        raise FtcError(rc, "ftc_launch_blocks")
    return out.value


def ftc_workspace_bytes(desc, S, is_allreduce=False) -> int:
    return load().ftc_workspace_bytes(C.byref(desc), S, int(is_allreduce))


def ftc_host_staging_bytes(desc, chunk_scenarios) -> int:
    return load().ftc_host_staging_bytes(C.byref(desc), chunk_scenarios)


def ftc_schedule_info(desc) -> dict:
    out = ftc_sched_t()
    rc = load().ftc_schedule_info(C.byref(desc), C.byref(out))
    if rc != FTC_OK:
        raise FtcError(rc, "ftc_schedule_info")
    return {n: getattr(out, n) for n, _ in ftc_sched_t._fields_}


def _batch(fn_name, desc, S, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace, stream, check):
    ws_bytes = 0 if d_workspace is None else d_workspace.numel() * d_workspace.element_size()
    rc = getattr(load(), fn_name)(C.byref(desc), S, _dev_ptr(d_in), _dev_ptr(d_prefail), _dev_ptr(d_inop),
                                  _dev_ptr(d_roots), _dev_ptr(d_out), _dev_ptr(d_status), _dev_ptr(d_workspace),
                                  ws_bytes, _stream(stream))
    if check and rc != FTC_OK:
        raise FtcError(rc, fn_name)
    return rc


def ftc_reduce_batch(desc, S, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace=None, stream=None,
                     check=True) -> int:
    return _batch("ftc_reduce_batch", desc, S, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace,
                  stream, check)


def ftc_allreduce_batch(desc, S, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace=None, stream=None,
                        check=True) -> int:
    return _batch("ftc_allreduce_batch", desc, S, d_in, d_prefail, d_inop, d_roots, d_out, d_status, d_workspace,
                  stream, check)


def ftc_reduce_batch_noalloc(desc, S, d_in, d_prefail, d_inop, d_roots, d_out, d_status, stream=None,
                             check=True) -> int:
    """Reduce on the library's built-in scratch array: for callers that can neither pass a workspace nor
    allocate one. Marshals the pointers only; no tensor is created here."""
    rc = load().ftc_reduce_batch_noalloc(C.byref(desc), S, _dev_ptr(d_in), _dev_ptr(d_prefail), _dev_ptr(d_inop),
                                         _dev_ptr(d_roots), _dev_ptr(d_out), _dev_ptr(d_status), _stream(stream))
    if check and rc != FTC_OK:
        raise FtcError(rc, "ftc_reduce_batch_noalloc")
    return rc


def ftc_candidates_kernel_name(desc) -> str:
    return load().ftc_candidates_kernel_name(C.byref(desc)).decode()


def ftc_candidates_workspace_bytes(desc, S) -> int:
    return load().ftc_candidates_workspace_bytes(C.byref(desc), S)


def ftc_candidates_batch(desc, S, is_allreduce, d_in, d_prefail, d_inop, d_roots, d_cand, d_cand_info, d_workspace,
                         stream=None, check=True) -> int:
    ws_bytes = 0 if d_workspace is None else d_workspace.numel() * d_workspace.element_size()
    rc = load().ftc_candidates_batch(C.byref(desc), S, int(is_allreduce), _dev_ptr(d_in), _dev_ptr(d_prefail),
                                     _dev_ptr(d_inop), _dev_ptr(d_roots), _dev_ptr(d_cand), _dev_ptr(d_cand_info),
                                     _dev_ptr(d_workspace), ws_bytes, _stream(stream))
    if check and rc != FTC_OK:
        raise FtcError(rc, "ftc_candidates_batch")
    return rc


def ftc_message_counts_batch(desc, S, is_allreduce, d_prefail, d_inop, d_roots, d_msgs, stream=None, check=True) -> int:
    rc = load().ftc_message_counts_batch(C.byref(desc), S, int(is_allreduce), _dev_ptr(d_prefail), _dev_ptr(d_inop),
                                         _dev_ptr(d_roots), _dev_ptr(d_msgs), _stream(stream))
    if check and rc != FTC_OK:
        raise FtcError(rc, "ftc_message_counts_batch")
    return rc


def ftc_failed_list_batch(desc, S, is_allreduce, d_prefail, d_inop, d_roots, d_failed, d_nfail, stream=None, check=True) -> int:
    rc = load().ftc_failed_list_batch(C.byref(desc), S, int(is_allreduce), _dev_ptr(d_prefail), _dev_ptr(d_inop),
                                      _dev_ptr(d_roots), _dev_ptr(d_failed), _dev_ptr(d_nfail), _stream(stream))
    if check and rc != FTC_OK:
        raise FtcError(rc, "ftc_failed_list_batch")
    return rc


def _batch_host(fn_name, desc, S, h_in, h_prefail, h_inop, h_roots, h_out, h_status, d_staging, stream, check):
    st_bytes = d_staging.numel() * d_staging.element_size()
    rc = getattr(load(), fn_name)(C.byref(desc), S, _host_ptr(h_in), _host_ptr(h_prefail), _host_ptr(h_inop),
                                  _host_ptr(h_roots), _host_ptr(h_out), _host_ptr(h_status), _dev_ptr(d_staging),
                                  st_bytes, _stream(stream))
    if check and rc != FTC_OK:
        raise FtcError(rc, fn_name)
    return rc


def ftc_reduce_batch_host(desc, S, h_in, h_prefail, h_inop, h_roots, h_out, h_status, d_staging, stream=None,
                          check=True) -> int:
    return _batch_host("ftc_reduce_batch_host", desc, S, h_in, h_prefail, h_inop, h_roots, h_out, h_status,
                       d_staging, stream, check)


def ftc_allreduce_batch_host(desc, S, h_in, h_prefail, h_inop, h_roots, h_out, h_status, d_staging, stream=None,
                             check=True) -> int:
    return _batch_host("ftc_allreduce_batch_host", desc, S, h_in, h_prefail, h_inop, h_roots, h_out, h_status,
                       d_staging, stream, check)


def ftc_read_bandwidth_probe(mode, d_buf, nbytes, d_sink, stream=None) -> int:
    rc = load().ftc_read_bandwidth_probe(mode, _dev_ptr(d_buf), nbytes, _dev_ptr(d_sink), _stream(stream))
    if rc != FTC_OK:
        raise FtcError(rc, "ftc_read_bandwidth_probe")
    return rc


def ftc_fill_inputs(kind, seed, first_scenario, S, P, k, d_out, stream=None) -> int:
    rc = load().ftc_fill_inputs(kind, seed & 0xFFFFFFFFFFFFFFFF, first_scenario, S, P, k, _dev_ptr(d_out),
                                _stream(stream))
    if rc != FTC_OK:
        raise FtcError(rc, "ftc_fill_inputs")
    return rc
