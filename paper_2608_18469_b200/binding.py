"""ctypes binding of the C ABI in include/erase.h: argument marshalling only.

Every function of the header is reachable under its own name through ``lib()``; ``Model`` is a
thin convenience wrapper that turns a spec dict (see ``synth``) into ``erase_model_spec`` and
numpy arrays into pointers.  Nothing of the training step is computed here: if the CUDA library
is missing or cannot be loaded this module raises; there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "liberase_b200.so")

OK, EINVAL, ENOMEM, ECUDA, ESTATE, ETIMEOUT, EUNSUPPORTED, ECOMM = range(8)
GRAPH, NO_OPT, EARLY_HEAD, BLOCK_OPT, SPLIT_BWD, STAMPS, PAR_FWD, PERSISTENT = 1, 2, 4, 8, 16, 32, 64, 128
LOCAL_GRADS = 256
COMM_ID_BYTES = 128
MAX_DIMS = 8

_DTYPE = {"f32": 0, "bf16": 1}
_INPUT = {"dense": 0, "tokens": 1, "ctr": 2}
_KIND = {"mlp": 0, "tower": 1, "transformer": 2, "cross": 3, "dot": 4, "main": 5}
_ACT = {"none": 0, "relu": 1, "gelu": 2}
_HEAD = {"bce": 0, "ce": 1, "goodness": 2}
_OPT = {"sgd": 0, "adam": 1, "adamw": 2}
_TOPO = {"chain": 0, "parallel": 1}


class BlockSpec(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_dims", C.c_int32), ("dims", C.c_int32 * MAX_DIMS),
                ("act", C.c_int32), ("n_heads", C.c_int32), ("n_cross", C.c_int32),
                ("head", C.c_int32), ("head_out", C.c_int32), ("flags", C.c_int32)]


class ModelSpec(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("input", C.c_int32), ("topo", C.c_int32), ("batch", C.c_int32),
                ("width", C.c_int32), ("seq", C.c_int32), ("vocab", C.c_int32), ("n_dense", C.c_int32),
                ("n_sparse", C.c_int32), ("table_rows", C.c_int32), ("emb_dim", C.c_int32),
                ("n_blocks", C.c_int32), ("blocks", C.POINTER(BlockSpec)), ("opt", C.c_int32),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("train_input", C.c_int32), ("replicas", C.c_int32),
                ("arena", C.c_void_p),
                ("arena_bytes", C.c_size_t)]


class Batch(C.Structure):
    _fields_ = [("x", C.c_void_p), ("ids", C.c_void_p), ("y", C.c_void_p)]


class OpRecord(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("block", C.c_int32), ("phase", C.c_int32),
                ("launches", C.c_int32), ("ms", C.c_float), ("flops", C.c_double), ("bytes", C.c_double)]


class EraseError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__(f"erase status {status}: {msg}")
        self.status = status


_lib = None

EXPORTS = {
    "erase_arena_bytes": (C.c_size_t, [C.POINTER(ModelSpec)]),
    "erase_create": (C.c_int, [C.POINTER(ModelSpec), C.POINTER(C.c_void_p)]),
    "erase_destroy": (None, [C.c_void_p]),
    "erase_num_tensors": (C.c_int32, [C.c_void_p]),
    "erase_tensor_info": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_char_p,
                                    C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_int32)]),
    "erase_set_params": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t]),
    "erase_params": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t]),
    "erase_grads": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t]),
    "erase_opt_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t,
                                  C.POINTER(C.c_int64)]),
    "erase_set_opt_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_int64]),
    "erase_step": (C.c_int, [C.c_void_p, C.POINTER(Batch), C.c_int32]),
    "erase_step_ex": (C.c_int, [C.c_void_p, C.POINTER(Batch), C.c_int32, C.c_uint32]),
    "erase_losses": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32]),
    "erase_sync": (C.c_int, [C.c_void_p]),
    "erase_selftest_timeout": (C.c_int, [C.c_void_p, C.c_int32]),
    "erase_comm_unique_id": (C.c_int, [C.c_void_p]),
    "erase_comm_init": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "erase_comm_order": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_int32)]),
    "erase_main_stream": (C.c_void_p, [C.c_void_p]),
    "erase_launch_count": (C.c_int64, [C.c_void_p]),
    "erase_timeline": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32]),
    "erase_gemm": (C.c_int, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_int64,
                             C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                             C.c_int32, C.c_void_p]),
    "erase_gemm_static": (C.c_int, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_int64,
                                    C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                                    C.c_int32, C.c_void_p]),
    "erase_gemm_static_error": (C.c_char_p, []),
    "erase_profile_step": (C.c_int, [C.c_void_p, C.POINTER(Batch), C.POINTER(OpRecord), C.c_int32,
                                     C.POINTER(C.c_int32)]),
    "erase_last_error": (C.c_char_p, [C.c_void_p]),
}


def lib():
    """The loaded shared library with argument types set.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_18469_b200.build`")
        _lib = C.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(_lib, name)
            fn.restype, fn.argtypes = res, args
    return _lib


def make_spec(spec, arena=None, arena_bytes=0):
    """spec dict -> (ModelSpec, keep-alive block array)."""
    blocks = (BlockSpec * len(spec["blocks"]))()
    for b, blk in zip(blocks, spec["blocks"]):
        b.kind = _KIND[blk["kind"]]
        b.n_dims = len(blk["dims"])
        for i, d in enumerate(blk["dims"]):
            b.dims[i] = d
        b.act = _ACT[blk.get("act", "none")]
        b.n_heads = blk.get("n_heads", 0)
        b.n_cross = blk.get("n_cross", 0)
        b.head = _HEAD[blk["head"]]
        b.head_out = blk["head_out"]
        b.flags = 1 if blk.get("reads_input") else 0
    o = spec["opt"]
    ms = ModelSpec(dtype=_DTYPE[spec["dtype"]], input=_INPUT[spec["input"]], topo=_TOPO[spec["topo"]],
                   batch=spec["batch"], width=spec["width"], seq=spec.get("seq", 0),
                   vocab=spec.get("vocab", 0), n_dense=spec.get("n_dense", 0),
                   n_sparse=spec.get("n_sparse", 0), table_rows=spec.get("table_rows", 0),
                   emb_dim=spec.get("emb_dim", 0), n_blocks=len(blocks),
                   blocks=C.cast(blocks, C.POINTER(BlockSpec)), opt=_OPT[o["kind"]], lr=o["lr"],
                   beta1=o.get("beta1", 0.9), beta2=o.get("beta2", 0.999), eps=o.get("eps", 1e-8),
                   weight_decay=o.get("wd", 0.0), train_input=1 if spec.get("train_input") else 0,
                   replicas=spec.get("replicas", 0), arena=arena, arena_bytes=arena_bytes)
    return ms, blocks


def comm_unique_id():
    """A fresh NCCL id (128 bytes) for erase_comm_init; make it on one replica and send it to the others."""
    buf = C.create_string_buffer(COMM_ID_BYTES)
    st = lib().erase_comm_unique_id(buf)
    if st != OK:
        raise EraseError(st, lib().erase_last_error(None).decode())
    return buf.raw


def _fptr(a):
    return a.ctypes.data_as(C.c_void_p)


class Model:
    """One model living on the current CUDA device.  Batches are device pointers (ints)."""

    def __init__(self, spec, arena=None, arena_bytes=0):
        self.spec = spec
        self._ms, self._blocks = make_spec(spec, arena, arena_bytes)
        h = C.c_void_p()
        st = lib().erase_create(C.byref(self._ms), C.byref(h))
        if st != OK:
            raise EraseError(st, lib().erase_last_error(None).decode())
        self.h = h
        self.n_blocks = len(spec["blocks"])

    def _ck(self, st):
        if st != OK:
            raise EraseError(st, lib().erase_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            lib().erase_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # tensors ---------------------------------------------------------------------------------
    def num_tensors(self):
        return lib().erase_num_tensors(self.h)

    def tensor_info(self, idx):
        blk, rank, tr = C.c_int32(), C.c_int32(), C.c_int32()
        name = C.create_string_buffer(32)
        shape = (C.c_int64 * 4)()
        self._ck(lib().erase_tensor_info(self.h, idx, C.byref(blk), name, C.byref(rank), shape, C.byref(tr)))
        return blk.value, name.value.decode(), tuple(shape[i] for i in range(rank.value)), bool(tr.value)

    def set_params(self, idx, arr):
        a = np.ascontiguousarray(arr, dtype=np.float32)
        self._ck(lib().erase_set_params(self.h, idx, _fptr(a), a.size))

    def set_all(self, flat):
        for i, a in enumerate(flat):
            self.set_params(i, a)

    def _get(self, fn, idx):
        shape = self.tensor_info(idx)[2]
        out = np.empty(shape, dtype=np.float32)
        self._ck(fn(self.h, idx, _fptr(out), out.size))
        return out

    def params(self, idx):
        return self._get(lib().erase_params, idx)

    def grads(self, idx):
        return self._get(lib().erase_grads, idx)

    def opt_state(self, idx):
        shape = self.tensor_info(idx)[2]
        m, v = np.empty(shape, np.float32), np.empty(shape, np.float32)
        t = C.c_int64()
        self._ck(lib().erase_opt_state(self.h, idx, _fptr(m), _fptr(v), m.size, C.byref(t)))
        return m, v, t.value

    def set_opt_state(self, idx, m, v, t):
        m = np.ascontiguousarray(m, np.float32)
        v = np.ascontiguousarray(v, np.float32)
        self._ck(lib().erase_set_opt_state(self.h, idx, _fptr(m), _fptr(v), m.size, t))

    # stepping ----------------------------------------------------------------------------------
    def step(self, x=None, ids=None, y=None, n_streams=1, flags=0):
        b = Batch(x=x, ids=ids, y=y)
        self._ck(lib().erase_step_ex(self.h, C.byref(b), n_streams, flags))

    def profile_step(self, x=None, ids=None, y=None, cap=4096):
        """One serial step with events around every operation -> list of dict records."""
        b = Batch(x=x, ids=ids, y=y)
        recs = (OpRecord * cap)()
        n = C.c_int32()
        self._ck(lib().erase_profile_step(self.h, C.byref(b), recs, cap, C.byref(n)))
        return [dict(name=r.name.decode(), block=r.block, phase=r.phase, launches=r.launches, ms=r.ms,
                     flops=r.flops, bytes=r.bytes) for r in recs[:min(n.value, cap)]]

    def losses(self):
        out = np.empty(self.n_blocks, np.float32)
        self._ck(lib().erase_losses(self.h, _fptr(out), self.n_blocks))
        return out

    def sync(self):
        self._ck(lib().erase_sync(self.h))

    def selftest_timeout(self, limit_us=1000):
        self._ck(lib().erase_selftest_timeout(self.h, limit_us))

    def comm_init(self, rank, world, unique_id):
        """Collective over the replicas: attach an NCCL communicator made from ``unique_id`` (128 bytes)."""
        buf = C.create_string_buffer(bytes(unique_id), COMM_ID_BYTES)
        self._ck(lib().erase_comm_init(self.h, rank, world, buf))

    def comm_order(self):
        """Block index of every exchange the last step enqueued, in order (-1: the losses)."""
        cap = self.n_blocks + 1
        out = (C.c_int32 * cap)()
        n = C.c_int32()
        self._ck(lib().erase_comm_order(self.h, out, cap, C.byref(n)))
        return [out[i] for i in range(min(n.value, cap))]

    def main_stream(self):
        return lib().erase_main_stream(self.h)

    def launch_count(self):
        return lib().erase_launch_count(self.h)

    def timeline(self):
        n = 2 * (2 * self.n_blocks + 1)
        out = np.empty(n, np.float32)
        self._ck(lib().erase_timeline(self.h, _fptr(out), n))
        return out.reshape(-1, 2)


def gemm(dtype, M, N, K, A, sa_m, sa_k, B, sb_n, sb_k, Cptr, ldc, c_f32=False, splits=1, engine=0, stream=None):
    """erase_gemm on device pointers (ints); raises EraseError on failure."""
    st = lib().erase_gemm(_DTYPE[dtype], M, N, K, A, sa_m, sa_k, B, sb_n, sb_k, Cptr, ldc, int(c_f32), splits,
                          engine, stream)
    if st != OK:
        raise EraseError(st, lib().erase_last_error(None).decode())


STATIC_WS_FLOATS = 2 * 1024 * 1024


def gemm_static(dtype, M, N, K, A, sa_m, sa_k, B, sb_n, sb_k, Cptr, ldc, c_f32=False, splits=1, engine=0,
                stream=None):
    """erase_gemm_static (no device allocation) on device pointers; raises EraseError on failure."""
    st = lib().erase_gemm_static(_DTYPE[dtype], M, N, K, A, sa_m, sa_k, B, sb_n, sb_k, Cptr, ldc, int(c_f32),
                                 splits, engine, stream)
    if st != OK:
        raise EraseError(st, lib().erase_gemm_static_error().decode())


def arena_bytes(spec):
    ms, _keep = make_spec(spec)
    return lib().erase_arena_bytes(C.byref(ms))
