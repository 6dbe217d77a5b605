"""ctypes binding of libadammini.so: argument marshalling only.

Every step of the Adam-mini update (Algorithm 1 of the paper) runs in the CUDA
library; this module converts Python arguments to the C ABI declared in
include/adammini.h and raises on error codes.  If the library has not been
built the first use raises: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Iterable, List, Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIBRARY = os.environ.get("ADAMMINI_LIBRARY") or os.path.join(_HERE, "libadammini.so")

WHOLE, ROWS, HEADS, TOKENS, FIXED, PART = 0, 1, 2, 3, 4, 5
F32, BF16 = 0, 1

(OPT_PATH, OPT_STREAM_CTAS, OPT_CLUSTER_SIZE, OPT_STREAM_THREADS, OPT_PROFILE, OPT_STREAM_CHUNK, OPT_CLUSTER_CHUNK,
 OPT_STATISTIC, OPT_STREAM_GROUPS, OPT_WAIT_LIMIT_US, OPT_TEST_STALL) = range(11)
STAT_MEAN, STAT_MAX, STAT_MIN, STAT_ONE_NORM, STAT_TWO_NORM = 0, 1, 2, 3, 4
(Q_LAUNCHES_PER_STEP, Q_SCRATCH_BYTES, Q_TOTAL_BLOCKS, Q_TOTAL_ELEMENTS, Q_ELEMENTS_SMALL,
 Q_ELEMENTS_STREAM, Q_ELEMENTS_CLUSTER, Q_ELEMENTS_TWOPASS, Q_ALGORITHMIC_BYTES, Q_BYTES_SMALL,
 Q_BYTES_STREAM, Q_BYTES_CLUSTER, Q_BYTES_TWOPASS, Q_STREAM_CTAS, Q_CLUSTER_SIZE, Q_CLUSTER_COUNT,
 Q_PART_TENSORS, Q_L2_BYTES, Q_SMEM_BYTES, Q_RESIDENT_CLUSTERS) = range(20)


class TensorDesc(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("cols", ctypes.c_int64), ("kind", ctypes.c_int32),
                ("n_heads", ctypes.c_int32), ("fixed_block_len", ctypes.c_int64),
                ("grad_dtype", ctypes.c_int32), ("apply_weight_decay", ctypes.c_int32)]


class TableRow(ctypes.Structure):
    _fields_ = [("numel", ctypes.c_int64), ("block_len", ctypes.c_int64), ("n_blocks", ctypes.c_int64),
                ("v_offset", ctypes.c_int64), ("kind", ctypes.c_int32), ("grad_dtype", ctypes.c_int32),
                ("wd", ctypes.c_int32), ("pad", ctypes.c_int32), ("mean_len", ctypes.c_int64)]


class HParams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_double), ("beta1", ctypes.c_double), ("beta2", ctypes.c_double),
                ("eps", ctypes.c_double), ("weight_decay", ctypes.c_double)]


class StepExtras(ctypes.Structure):
    _fields_ = [("params_bf16", ctypes.POINTER(ctypes.c_void_p)), ("grad_scale", ctypes.c_double),
                ("grad_scale_device", ctypes.c_void_p), ("skip_flag", ctypes.c_void_p),
                ("part_sums", ctypes.c_void_p)]


class AdamMiniError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"adammini: {message} (status {status})")
        self.status = status


_lib: Optional[ctypes.CDLL] = None

_SIGNATURES = {
    "adammini_partition_build": (ctypes.c_int, [ctypes.POINTER(TensorDesc), ctypes.c_int32, ctypes.POINTER(ctypes.c_void_p)]),
    "adammini_partition_num_tensors": (ctypes.c_int32, [ctypes.c_void_p]),
    "adammini_partition_export": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(TableRow), ctypes.POINTER(ctypes.c_int64)]),
    "adammini_partition_free": (None, [ctypes.c_void_p]),
    "adammini_kind_from_name": (ctypes.c_int32, [ctypes.c_char_p]),
    "adammini_create": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(HParams), ctypes.POINTER(ctypes.c_void_p)]),
    "adammini_set_lr": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_double]),
    "adammini_set_hparams": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(HParams)]),
    "adammini_step": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p),
                                     ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]),
    "adammini_step_ex": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p),
                                        ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                        ctypes.POINTER(StepExtras)]),
    "adammini_part_sums": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, ctypes.c_void_p]),
    "adammini_probe_ring_copy": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
                                                ctypes.c_int32, ctypes.c_void_p]),
    "adammini_step_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p),
                                          ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64]),
    "adammini_step_tensor_noalloc": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                    ctypes.c_int64, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32,
                                                    ctypes.POINTER(HParams), ctypes.c_int64, ctypes.c_void_p]),
    "adammini_sync_status": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "adammini_set_option": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64]),
    "adammini_query": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int64)]),
    "adammini_choose_cluster_size": (ctypes.c_int32, [ctypes.POINTER(ctypes.c_int32), ctypes.c_int64, ctypes.c_int64]),
    "adammini_get_profile": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]),
    "adammini_last_cuda_error": (ctypes.c_int, [ctypes.c_void_p]),
    "adammini_destroy": (ctypes.c_int, [ctypes.c_void_p]),
    "adammini_status_string": (ctypes.c_char_p, [ctypes.c_int]),
}


def exported_names() -> List[str]:
    """Names of the entry points this binding expects the library to export."""
    return sorted(_SIGNATURES)


def load() -> ctypes.CDLL:
    """Load libadammini.so (built in-tree by paper_2406_16793_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIBRARY):
            raise RuntimeError(
                f"{LIBRARY} is missing: build it with `python -m paper_2406_16793_b200.build` "
                "(there is no CPU fallback)")
        lib = ctypes.CDLL(LIBRARY)
        for name, (res, args) in _SIGNATURES.items():
            try:
                fn = getattr(lib, name)
            except AttributeError:
                if os.environ.get("ADAMMINI_LIBRARY"):
                    continue            # an older build named explicitly: its missing calls fail when used
                raise
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def _check(status: int, handle=None) -> None:
    if status != 0:
        lib = load()
        msg = lib.adammini_status_string(status).decode()
        if status == -4:          # no handle: the error of the creation that just failed
            msg += f" (cudaError {lib.adammini_last_cuda_error(handle)})"
        raise AdamMiniError(status, msg)


def kind_from_name(name: str) -> int:
    """Algorithm 3's name tests (embed/output, query/key, value/attn.proj/mlp, else)."""
    return int(load().adammini_kind_from_name(name.encode()))


def choose_cluster_size(resident_clusters: Sequence[int], l2_bytes: int, block_bytes: int) -> int:
    """The library's choice of CTAs per cluster for head-sized blocks (host logic only):
    resident_clusters[c] = clusters of c CTAs the device keeps resident, c = 1..8 (entry 0 unused)."""
    arr = (ctypes.c_int32 * 9)(*([0] * 9))
    for c, n in enumerate(list(resident_clusters)[:9]):
        arr[c] = int(n)
    return int(load().adammini_choose_cluster_size(arr, int(l2_bytes), int(block_bytes)))


NOALLOC_MAX_BLOCKS = 32768
NOALLOC_MAX_PIECES = 32768


def step_tensor_noalloc(param, grad, m, v, block_len: int, step: int, *, lr: float = 1e-3, beta1: float = 0.9,
                        beta2: float = 0.95, eps: float = 1e-8, weight_decay: float = 0.1,
                        apply_weight_decay: bool = True, stream: int = 0) -> None:
    """One Adam-mini step on one tensor through the entry point that allocates
    nothing (for callers that may not call cudaMalloc: allocator callbacks,
    loops whose memory pool owns the device, latency-critical sections).  The
    tensors are device tensors; v has numel/block_len entries.  All calls on a
    device share one fixed scratch array inside the library, so issue them on
    one stream (or order them); at most NOALLOC_MAX_BLOCKS blocks per call."""
    numel = int(param.numel())
    dtype = BF16 if str(grad.dtype) == "torch.bfloat16" else F32
    hp = HParams(lr, beta1, beta2, eps, weight_decay)
    _check(load().adammini_step_tensor_noalloc(
        int(param.data_ptr()), int(grad.data_ptr()), int(m.data_ptr()), int(v.data_ptr()), numel,
        int(block_len), dtype, int(bool(apply_weight_decay)), ctypes.byref(hp), int(step), stream or None))


class Partition:
    """Flat block table built by the library's host partitioner."""

    def __init__(self, descs: Iterable):
        """`descs`: objects with rows, cols, kind, n_heads, fixed_block_len,
        grad_dtype, apply_weight_decay attributes (e.g. workloads.TensorSpec)."""
        lib = load()
        items = list(descs)
        arr = (TensorDesc * max(len(items), 1))()
        for i, d in enumerate(items):
            arr[i] = TensorDesc(int(d.rows), int(d.cols), int(d.kind), int(getattr(d, "n_heads", 0)),
                                int(getattr(d, "fixed_block_len", 0)), int(d.grad_dtype),
                                int(getattr(d, "apply_weight_decay", 1)))
        self._ptr = ctypes.c_void_p()
        _check(lib.adammini_partition_build(arr, len(items), ctypes.byref(self._ptr)))
        self.n_tensors = int(lib.adammini_partition_num_tensors(self._ptr))

    def export(self):
        """Returns (list of TableRow, total_blocks)."""
        lib = load()
        rows = (TableRow * max(self.n_tensors, 1))()
        total = ctypes.c_int64()
        _check(lib.adammini_partition_export(self._ptr, rows, ctypes.byref(total)))
        return [rows[i] for i in range(self.n_tensors)], int(total.value)

    @property
    def total_blocks(self) -> int:
        return self.export()[1]

    def close(self) -> None:
        if self._ptr:
            load().adammini_partition_free(self._ptr)
            self._ptr = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _ptr_array(ptrs: Sequence[int]):
    arr = (ctypes.c_void_p * max(len(ptrs), 1))()
    for i, p in enumerate(ptrs):
        arr[i] = p
    return arr


def _data_ptrs(tensors: Sequence) -> List[int]:
    return [int(t.data_ptr()) if hasattr(t, "data_ptr") else int(t) for t in tensors]


class AdamMini:
    """Optimizer handle on the current CUDA device."""

    def __init__(self, partition: Partition, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.95,
                 eps: float = 1e-8, weight_decay: float = 0.1):
        lib = load()
        self._h = ctypes.c_void_p()
        hp = HParams(lr, beta1, beta2, eps, weight_decay)
        _check(lib.adammini_create(partition._ptr, ctypes.byref(hp), ctypes.byref(self._h)))
        self.n_tensors = partition.n_tensors
        self._cached = None

    def set_lr(self, lr: float) -> None:
        _check(load().adammini_set_lr(self._h, float(lr)), self._h)

    def set_hparams(self, lr, beta1, beta2, eps, weight_decay) -> None:
        hp = HParams(lr, beta1, beta2, eps, weight_decay)
        _check(load().adammini_set_hparams(self._h, ctypes.byref(hp)), self._h)

    def set_option(self, key: int, value: int) -> None:
        _check(load().adammini_set_option(self._h, int(key), int(value)), self._h)

    def query(self, what: int) -> int:
        out = ctypes.c_int64()
        _check(load().adammini_query(self._h, int(what), ctypes.byref(out)), self._h)
        return int(out.value)

    def _arrays(self, params, grads, m):
        key = (tuple(_data_ptrs(params)), tuple(_data_ptrs(grads)), tuple(_data_ptrs(m)))
        if self._cached is None or self._cached[0] != key:
            if not (len(key[0]) == len(key[1]) == len(key[2]) == self.n_tensors):
                raise ValueError("params, grads and m must each have one entry per tensor of the partition")
            self._cached = (key, _ptr_array(key[0]), _ptr_array(key[1]), _ptr_array(key[2]))
        return self._cached[1:]

    def step(self, params: Sequence, grads: Sequence, m: Sequence, v, step: int, stream: int = 0) -> None:
        """One Adam-mini step.  params/grads/m: device tensors (or raw device
        addresses) in table order; v: device float32[total_blocks]; `stream`: a
        raw cudaStream_t (0 = default stream).  Asynchronous."""
        pa, ga, ma = self._arrays(params, grads, m)
        vp = int(v.data_ptr()) if hasattr(v, "data_ptr") else int(v)
        _check(load().adammini_step(self._h, pa, ga, ma, vp, int(step), stream or None), self._h)

    def step_ex(self, params: Sequence, grads: Sequence, m: Sequence, v, step: int, stream: int = 0, *,
                params_bf16: Optional[Sequence] = None, grad_scale: float = 1.0, grad_scale_device=None,
                skip_flag=None, part_sums=None) -> None:
        """A step with the optional extras of adammini_step_ex: bf16 copies of the
        updated parameters, a gradient scale (host value and/or device scalar)
        and a device flag that turns the step into a no-op."""
        pa, ga, ma = self._arrays(params, grads, m)
        vp = int(v.data_ptr()) if hasattr(v, "data_ptr") else int(v)
        ex = StepExtras()
        keep = None
        if params_bf16 is not None:
            keep = _ptr_array([0 if t is None else (int(t.data_ptr()) if hasattr(t, "data_ptr") else int(t))
                               for t in params_bf16])
            ex.params_bf16 = ctypes.cast(keep, ctypes.POINTER(ctypes.c_void_p))
        ex.grad_scale = float(grad_scale)
        ex.grad_scale_device = int(grad_scale_device.data_ptr()) if grad_scale_device is not None else None
        ex.skip_flag = int(skip_flag.data_ptr()) if skip_flag is not None else None
        ex.part_sums = int(part_sums.data_ptr()) if part_sums is not None else None
        _check(load().adammini_step_ex(self._h, pa, ga, ma, vp, int(step), stream or None, ctypes.byref(ex)), self._h)

    def part_sums(self, grads: Sequence, out, stream: int = 0) -> None:
        """Sums of g*g of this holder's parts of cut blocks (the table's PART
        tensors, in table order) into `out`, a device float64 tensor."""
        ga = _ptr_array(_data_ptrs(grads))
        _check(load().adammini_part_sums(self._h, ga, int(out.data_ptr()), stream or None), self._h)

    def probe_ring_copy(self, src, dst, n_items: int, load_bytes: int, store_bytes: int, stream: int = 0) -> None:
        """Measurement aid: a copy through the streaming kernel's ring with no arithmetic
        (item i reads load_bytes at src + i * load_bytes and writes store_bytes at
        dst + i * store_bytes).  src/dst: device tensors, raw addresses or None.  Asynchronous."""
        sp = 0 if src is None else (int(src.data_ptr()) if hasattr(src, "data_ptr") else int(src))
        dp = 0 if dst is None else (int(dst.data_ptr()) if hasattr(dst, "data_ptr") else int(dst))
        _check(load().adammini_probe_ring_copy(self._h, sp or None, dp or None, int(n_items), int(load_bytes), int(store_bytes),
                                               stream or None), self._h)

    def step_host(self, params: Sequence, grads: Sequence, m: Sequence, v, step: int,
                  staging_bytes: int = 0) -> None:
        """The same step with params/grads/m/v in HOST memory (CPU tensors or raw
        host addresses); returns when the results are back in host memory."""
        pa, ga, ma = _ptr_array(_data_ptrs(params)), _ptr_array(_data_ptrs(grads)), _ptr_array(_data_ptrs(m))
        vp = int(v.data_ptr()) if hasattr(v, "data_ptr") else int(v)
        _check(load().adammini_step_host(self._h, pa, ga, ma, vp, int(step), int(staging_bytes)), self._h)

    def get_profile(self):
        """Mean device milliseconds per step of each kernel family over the steps
        recorded since OPT_PROFILE was set: ([short-block, streaming, cluster,
        two-pass], number of steps averaged)."""
        ms = (ctypes.c_float * 4)()
        n = ctypes.c_int32()
        _check(load().adammini_get_profile(self._h, ms, ctypes.byref(n)), self._h)
        return [float(x) for x in ms], int(n.value)

    def sync_status(self, stream: int = 0) -> None:
        """Wait for the stream; raises if a device-side bounded wait gave up."""
        _check(load().adammini_sync_status(self._h, stream or None), self._h)

    def close(self) -> None:
        if self._h:
            load().adammini_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
