"""Thin ctypes binding of libgcnsa (argument marshalling only).

Every step of the training path runs in the library's CUDA kernels.  PyTorch
is used for device memory (its caching allocator serves the library's
``alloc`` / ``free`` callbacks) and for the stream the work is enqueued on.
There is no CPU fallback: if the shared library is missing, loading fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgcnsa.so")

PART_RANGE, PART_HASH, PART_USER = 0, 1, 2
BUILD_DEVICE, BUILD_HOST = 0, 1
GEMM_FP32, GEMM_TF32X3, GEMM_TF32 = 0, 1, 2
AGG_GRAD_AVG, AGG_PARAM_AVG = 0, 1
EPI_NONE, EPI_BIAS, EPI_BIAS_RELU, EPI_MASK, EPI_ROWSCALE = 0, 1, 2, 3, 4
MAX_LAYERS = 8
(GET_W, GET_B, GET_GRAD_W, GET_GRAD_B, GET_ADAM_M_W, GET_ADAM_M_B, GET_ADAM_V_W, GET_ADAM_V_B, GET_ACT,
 GET_DLOGITS) = range(10)

ERR_ARG, ERR_NOT_SYMMETRIC, ERR_SELF_LOOP_OR_DUP, ERR_LABEL_RANGE, ERR_OOM, ERR_ORDER, ERR_CUDA, ERR_ARCH, ERR_TOO_LARGE = (
    -1, -2, -3, -4, -5, -6, -7, -8, -9)

ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class Env(C.Structure):
    _fields_ = [("alloc", ALLOC_FN), ("free", FREE_FN), ("user", C.c_void_p), ("stream", C.c_void_p),
                ("device", C.c_int32)]


class Graph(C.Structure):
    _fields_ = [("n", C.c_int64), ("nnz", C.c_int64), ("rowptr", C.c_void_p), ("col", C.c_void_p),
                ("f", C.c_int32), ("x", C.c_void_p), ("ldx", C.c_int64), ("c", C.c_int32), ("y", C.c_void_p),
                ("train_mask", C.c_void_p)]


class PartOpts(C.Structure):
    _fields_ = [("m", C.c_int32), ("overlap_ppm", C.c_uint32), ("seed", C.c_uint64), ("part_mode", C.c_int32),
                ("user_part", C.c_void_p), ("loss_on_halo", C.c_int32), ("builder", C.c_int32), ("order_window", C.c_int32)]


class PartInfo(C.Structure):
    _fields_ = [("n_owned", C.c_int64), ("n_halo", C.c_int64), ("n", C.c_int64), ("nnz", C.c_int64),
                ("nts", C.c_int64), ("n_train", C.c_int64), ("max_depth", C.c_int32)]


class PartHost(C.Structure):
    _fields_ = [("rowptr", C.c_void_p), ("col", C.c_void_p), ("val", C.c_void_p), ("t_rowptr", C.c_void_p),
                ("t_col", C.c_void_p), ("t_val", C.c_void_p), ("members", C.c_void_p), ("depth", C.c_void_p)]


class PartScheduleHost(C.Structure):
    _fields_ = [("order", C.c_void_p), ("t_order", C.c_void_p), ("m_order", C.c_void_p), ("tm_rowptr", C.c_void_p),
                ("tm_col", C.c_void_p), ("tm_order", C.c_void_p), ("mask", C.c_void_p), ("y", C.c_void_p)]


class PartScheduleInfo(C.Structure):
    _fields_ = [("n_long", C.c_int64), ("t_n_long", C.c_int64), ("m_n_long", C.c_int64), ("tm_n_long", C.c_int64),
                ("m_nnz", C.c_int64), ("tm_nnz", C.c_int64)]


class ModelOpts(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("dims", C.c_int32 * (MAX_LAYERS + 1)), ("use_bias", C.c_int32),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("gemm_mode", C.c_int32), ("agg_mode", C.c_int32), ("loss_rows_only", C.c_int32), ("epoch_graph", C.c_int32),
                ("factored_norm", C.c_int32), ("cache_ax", C.c_int32)]


class SageOpts(C.Structure):
    _fields_ = [("dims", C.c_int32 * 3), ("fanout", C.c_int32 * 2), ("batch", C.c_int32), ("lr", C.c_float),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("seed", C.c_uint64),
                ("gemm_mode", C.c_int32), ("batch_graph", C.c_int32)]


class SageBatchHost(C.Structure):
    _fields_ = [("vertices", C.c_void_p), ("count2", C.c_void_p), ("samples1", C.c_void_p), ("count1", C.c_void_p),
                ("hidden", C.c_void_p), ("logits", C.c_void_p), ("dlogits", C.c_void_p), ("loss", C.c_void_p)]


class Profile(C.Structure):
    _fields_ = [("ms", C.c_double * 3), ("launches", C.c_int64 * 3), ("alg_bytes", C.c_double * 3),
                ("flops", C.c_double * 3), ("l1_bytes", C.c_double * 3), ("alg_bytes_val", C.c_double * 3)]


class GcnsaError(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"gcnsa error {code}: {text}")
        self.code = code


_lib = None

_SIGS = {
    "gcnsa_strerror": (C.c_char_p, [C.c_int]),
    "gcnsa_last_error": (C.c_char_p, []),
    "gcnsa_launch_count": (C.c_int64, []),
    "gcnsa_gemm_path_counts": (C.c_int, [C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "gcnsa_model_opts_default": (None, [C.POINTER(ModelOpts)]),
    "gcnsa_tc_clear": (C.c_int, []),
    "gcnsa_debug_status": (C.c_int, [C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int64)]),
    "gcnsa_build_partitions": (C.c_int, [C.POINTER(Env), C.POINTER(Graph), C.POINTER(PartOpts), C.POINTER(C.c_void_p)]),
    "gcnsa_plan_create": (C.c_int, [C.POINTER(Graph), C.POINTER(PartOpts), C.POINTER(C.c_void_p)]),
    "gcnsa_plan_info": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(PartInfo)]),
    "gcnsa_plan_assignment": (C.c_int, [C.c_void_p, C.c_void_p]),
    "gcnsa_plan_export": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(PartHost)]),
    "gcnsa_plan_export_schedule": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(PartScheduleInfo),
                                             C.POINTER(PartScheduleHost)]),
    "gcnsa_plan_destroy": (C.c_int, [C.c_void_p]),
    "gcnsa_parts_count": (C.c_int, [C.c_void_p]),
    "gcnsa_parts_info": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(PartInfo)]),
    "gcnsa_parts_assignment": (C.c_int, [C.c_void_p, C.c_void_p]),
    "gcnsa_parts_export": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(PartHost)]),
    "gcnsa_parts_export_schedule": (C.c_int, [C.c_void_p, C.c_int32, C.POINTER(PartScheduleInfo),
                                              C.POINTER(PartScheduleHost)]),
    "gcnsa_parts_get_features": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]),
    "gcnsa_parts_set_features": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p]),
    "gcnsa_parts_destroy": (C.c_int, [C.c_void_p]),
    "gcnsa_model_create": (C.c_int, [C.POINTER(Env), C.c_void_p, C.POINTER(ModelOpts), C.POINTER(C.c_void_p),
                                     C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]),
    "gcnsa_forward": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]),
    "gcnsa_backward": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32]),
    "gcnsa_step": (C.c_int, [C.c_void_p]),
    "gcnsa_epoch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "gcnsa_epoch_host": (C.c_int, [C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p), C.c_void_p]),
    "gcnsa_model_get": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t]),
    "gcnsa_model_set": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t]),
    "gcnsa_model_profile": (C.c_int, [C.c_void_p, C.c_int32]),
    "gcnsa_model_profile_read": (C.c_int, [C.c_void_p, C.c_void_p]),
    "gcnsa_evaluate": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(C.c_int64),
                                 C.POINTER(C.c_int64), C.c_void_p]),
    "gcnsa_model_copy_params": (C.c_int, [C.c_void_p, C.c_void_p]),
    "gcnsa_model_select_partition": (C.c_int, [C.c_void_p, C.c_int32]),
    "gcnsa_model_get_t": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64)]),
    "gcnsa_model_set_t": (C.c_int, [C.c_void_p, C.c_int64]),
    "gcnsa_model_destroy": (C.c_int, [C.c_void_p]),
    "gcnsa_sage_create": (C.c_int, [C.POINTER(Env), C.c_void_p, C.POINTER(SageOpts), C.POINTER(C.c_void_p),
                                    C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]),
    "gcnsa_sage_epoch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "gcnsa_sage_get_epoch": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64)]),
    "gcnsa_sage_profile": (C.c_int, [C.c_void_p, C.c_int32]),
    "gcnsa_sage_profile_read": (C.c_int, [C.c_void_p, C.c_void_p]),
    "gcnsa_sage_batches": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int64)]),
    "gcnsa_sage_batch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int64, C.c_int64, C.c_int32, C.c_void_p]),
    "gcnsa_sage_batch_shape": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "gcnsa_sage_batch_export": (C.c_int, [C.c_void_p, C.POINTER(SageBatchHost)]),
    "gcnsa_sage_get": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_size_t]),
    "gcnsa_sage_destroy": (C.c_int, [C.c_void_p]),
    "gcnsa_op_spmm": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p,
                                C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64]),
    "gcnsa_op_spmm_pattern": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p,
                                        C.c_int64]),
    "gcnsa_op_gemm": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_int64,
                                C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int32,
                                C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t]),
    "gcnsa_op_gemm_workspace": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_int64]),
    "gcnsa_op_gemm_mask_colsum": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_int64,
                                            C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                            C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                            C.c_size_t, C.c_void_p, C.c_size_t]),
    "gcnsa_op_gemm_mask_colsum_scratch": (C.c_size_t, [C.c_int64, C.c_int32]),
    "gcnsa_tc_status": (C.c_int, [C.POINTER(C.c_int32)]),
    "gcnsa_op_gather_probe": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_void_p, C.c_size_t]),
    "gcnsa_op_gather_probe_warps": (C.c_int, [C.POINTER(C.c_int32)]),
    "gcnsa_op_softmax_ce": (C.c_int, [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p,
                                      C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t]),
    "gcnsa_op_softmax_ce_scratch": (C.c_size_t, [C.c_int64]),
    "gcnsa_op_colsum": (C.c_int, [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32,
                                  C.c_void_p, C.c_size_t]),
    "gcnsa_op_colsum_scratch": (C.c_size_t, [C.c_int64, C.c_int32]),
    "gcnsa_op_colsum_scaled": (C.c_int, [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32,
                                         C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_int64]),
    "gcnsa_op_colsum_static": (C.c_int, [C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32]),
    "gcnsa_op_adam": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                C.c_float, C.c_float, C.c_float, C.c_float, C.c_int64]),
    "gcnsa_op_normalize": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
}


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; "
                              "g.build()'` (there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGS.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def exported_symbols():
    return sorted(_SIGS)


def _ck(rc):
    if rc != 0:
        L = lib()
        raise GcnsaError(rc, f"{L.gcnsa_strerror(rc).decode()}: {L.gcnsa_last_error().decode()}")


def launch_count() -> int:
    return int(lib().gcnsa_launch_count())


def gemm_path_counts() -> tuple:
    """(tensor_core, fp32_fallback): dense products asked for in GEMM_TF32X3 mode that the tcgen05 kernel took,
    and those that ran on the fp32 FMA kernel instead."""
    a, b = C.c_int64(), C.c_int64()
    _ck(lib().gcnsa_gemm_path_counts(C.byref(a), C.byref(b)))
    return int(a.value), int(b.value)


# The option set the published throughput figures belong to (what gcnsa_model_opts_default fills in, and the
# defaults of Model below), and the plainest path (what a zeroed gcnsa_model_opts selects).
MEASURED = dict(gemm_mode=GEMM_TF32X3, loss_rows_only=1, epoch_graph=1, factored_norm=1)
PLAIN = dict(gemm_mode=GEMM_FP32, loss_rows_only=0, epoch_graph=0, factored_norm=0)


# --------------------------------------------------------- memory + stream ---
_torch_fns = {"alloc": None, "delete": None, "stream": None}


@ALLOC_FN
def _torch_alloc(nbytes, user):
    try:
        return _torch_fns["alloc"](int(nbytes), stream=_torch_fns["stream"]())
    except Exception:  # noqa: BLE001 - reported to the caller as a NULL pointer
        return None


@FREE_FN
def _torch_free(ptr, user):
    fn = _torch_fns["delete"] if _torch_fns is not None else None
    if fn is not None:   # at interpreter shutdown the allocator is already gone
        try:
            fn(ptr)
        except Exception:  # noqa: BLE001
            pass


def make_env(device: int = 0, stream=None, torch_memory: bool = True) -> Env:
    """Environment whose memory comes from torch's caching allocator and whose
    stream is torch's current stream (or the one given)."""
    import torch
    _torch_fns.update(alloc=torch.cuda.caching_allocator_alloc, delete=torch.cuda.caching_allocator_delete,
                      stream=torch.cuda.current_stream)
    if stream is None:
        stream = torch.cuda.current_stream(device)
    env = Env()
    if torch_memory:
        env.alloc, env.free = _torch_alloc, _torch_free
    env.user = None
    env.stream = stream.cuda_stream
    env.device = device
    return env


def _np(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def _hp(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _graph_args(rowptr, col, x, y, train_mask, n_classes, m, overlap_ppm, seed, part_mode, user_part, loss_on_halo,
                builder=BUILD_DEVICE, order_window=0):
    rowptr, col = _np(rowptr, np.int64), _np(col, np.int32)
    x, y, train_mask = _np(x, np.float32), _np(y, np.int32), _np(train_mask, np.uint8)
    f = x.shape[1] if x.ndim == 2 else 0
    g = Graph(n=rowptr.size - 1, nnz=col.size, rowptr=_hp(rowptr), col=_hp(col), f=f, x=_hp(x), ldx=f, c=n_classes,
              y=_hp(y), train_mask=_hp(train_mask))
    up = None if user_part is None else _np(user_part, np.int32)
    o = PartOpts(m=m, overlap_ppm=overlap_ppm, seed=seed, part_mode=part_mode, user_part=_hp(up),
                 loss_on_halo=loss_on_halo, builder=builder, order_window=order_window)
    return g, o, (rowptr, col, x, y, train_mask, up)  # the arrays must outlive the call


class Plan:
    """Host-only result of the master step: assignment, Algorithm 1 and the
    structure of every extended partition.  Needs no GPU."""

    def __init__(self, rowptr, col, x, y, train_mask, n_classes, m, overlap_ppm, seed, part_mode=PART_RANGE,
                 user_part=None, loss_on_halo=1, order_window=0):
        g, o, keep = _graph_args(rowptr, col, x, y, train_mask, n_classes, m, overlap_ppm, seed, part_mode, user_part,
                                 loss_on_halo, order_window=order_window)
        self.handle = C.c_void_p()
        _ck(lib().gcnsa_plan_create(C.byref(g), C.byref(o), C.byref(self.handle)))
        self.m, self.n = m, int(g.n)

    def info(self, p) -> PartInfo:
        out = PartInfo()
        _ck(lib().gcnsa_plan_info(self.handle, p, C.byref(out)))
        return out

    def assignment(self) -> np.ndarray:
        part = np.empty(self.n, dtype=np.int32)
        _ck(lib().gcnsa_plan_assignment(self.handle, _hp(part)))
        return part

    def export(self, p) -> dict:
        i = self.info(p)
        out = {"rowptr": np.empty(i.n + 1, np.int32), "col": np.empty(i.nnz, np.int32),
               "t_rowptr": np.empty(i.n + 1, np.int32), "t_col": np.empty(i.nnz, np.int32),
               "members": np.empty(i.n, np.int64), "depth": np.empty(self.m, np.int32)}
        h = PartHost(**{k: _hp(v) for k, v in out.items()})
        _ck(lib().gcnsa_plan_export(self.handle, p, C.byref(h)))
        return out

    def export_schedule(self, p) -> dict:
        """Row orders, loss rows and the transposed CSR over the loss columns as the host builder makes them."""
        i = self.info(p)
        si = PartScheduleInfo()
        _ck(lib().gcnsa_plan_export_schedule(self.handle, p, C.byref(si), None))
        out = {"order": np.empty(i.n, np.int32), "t_order": np.empty(i.n, np.int32),
               "m_order": np.empty(i.n_train, np.int32), "tm_rowptr": np.empty(i.n + 1, np.int32),
               "tm_col": np.empty(si.tm_nnz, np.int32), "tm_order": np.empty(i.n, np.int32)}
        h = PartScheduleHost(**{k: _hp(v) for k, v in out.items()})
        _ck(lib().gcnsa_plan_export_schedule(self.handle, p, C.byref(si), C.byref(h)))
        for k in ("n_long", "t_n_long", "m_n_long", "tm_n_long", "m_nnz", "tm_nnz"):
            out[k] = int(getattr(si, k))
        return out

    def close(self):
        if self.handle:
            lib().gcnsa_plan_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:  # noqa: BLE001
            pass


class Parts:
    """All extended partitions of one graph, resident on the device."""

    def __init__(self, env: Env, rowptr, col, x, y, train_mask, n_classes, m, overlap_ppm, seed,
                 part_mode=PART_RANGE, user_part=None, loss_on_halo=1, builder=BUILD_DEVICE, order_window=0):
        g, o, keep = _graph_args(rowptr, col, x, y, train_mask, n_classes, m, overlap_ppm, seed, part_mode, user_part,
                                 loss_on_halo, builder, order_window)
        self.env = env
        self.handle = C.c_void_p()
        _ck(lib().gcnsa_build_partitions(C.byref(env), C.byref(g), C.byref(o), C.byref(self.handle)))
        self.m, self.n, self.f, self.c = m, int(g.n), int(g.f), n_classes

    def info(self, p) -> PartInfo:
        out = PartInfo()
        _ck(lib().gcnsa_parts_info(self.handle, p, C.byref(out)))
        return out

    def assignment(self) -> np.ndarray:
        part = np.empty(self.n, dtype=np.int32)
        _ck(lib().gcnsa_parts_assignment(self.handle, _hp(part)))
        return part

    def export(self, p) -> dict:
        i = self.info(p)
        out = {"rowptr": np.empty(i.n + 1, np.int32), "col": np.empty(i.nnz, np.int32), "val": np.empty(i.nnz, np.float32),
               "t_rowptr": np.empty(i.n + 1, np.int32), "t_col": np.empty(i.nnz, np.int32),
               "t_val": np.empty(i.nnz, np.float32), "members": np.empty(i.n, np.int64), "depth": np.empty(self.m, np.int32)}
        h = PartHost(**{k: _hp(v) for k, v in out.items()})
        _ck(lib().gcnsa_parts_export(self.handle, p, C.byref(h)))
        return out

    def export_schedule(self, p) -> dict:
        """The library's scheduling structures of partition p (row orders, loss rows, the transposed CSR over
        the loss columns) and the counts that go with them."""
        i = self.info(p)
        si = PartScheduleInfo()
        _ck(lib().gcnsa_parts_export_schedule(self.handle, p, C.byref(si), None))
        out = {"order": np.empty(i.n, np.int32), "t_order": np.empty(i.n, np.int32),
               "m_order": np.empty(i.n_train, np.int32), "tm_rowptr": np.empty(i.n + 1, np.int32),
               "tm_col": np.empty(si.tm_nnz, np.int32), "tm_order": np.empty(i.n, np.int32),
               "mask": np.empty(i.n, np.uint8), "y": np.empty(i.n, np.int32)}
        h = PartScheduleHost(**{k: _hp(v) for k, v in out.items()})
        _ck(lib().gcnsa_parts_export_schedule(self.handle, p, C.byref(si), C.byref(h)))
        for k in ("n_long", "t_n_long", "m_n_long", "tm_n_long", "m_nnz", "tm_nnz"):
            out[k] = int(getattr(si, k))
        return out

    def features(self, p) -> np.ndarray:
        i = self.info(p)
        x = np.empty((i.n, self.f), np.float32)
        _ck(lib().gcnsa_parts_get_features(self.handle, p, _hp(x)))
        return x

    def members(self, p) -> np.ndarray:
        i = self.info(p)
        mem = np.empty(i.n, np.int64)
        h = PartHost(members=_hp(mem))
        _ck(lib().gcnsa_parts_export(self.handle, p, C.byref(h)))
        return mem

    def set_features(self, p, x_host_ptr):
        _ck(lib().gcnsa_parts_set_features(self.handle, p, x_host_ptr))

    def close(self):
        if self.handle:
            lib().gcnsa_parts_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:  # noqa: BLE001
            pass


class Model:
    """Weights, Adam state, gradient sum and work buffers for one set of partitions."""

    def __init__(self, env: Env, parts: Parts, dims, w0, b0=None, use_bias=1, lr=0.02, beta1=0.9, beta2=0.999,
                 eps=1e-8, gemm_mode=GEMM_TF32X3, agg_mode=AGG_GRAD_AVG, loss_rows_only=1, epoch_graph=1,
                 factored_norm=1, cache_ax=0):
        L = len(dims) - 1
        o = ModelOpts(n_layers=L, use_bias=use_bias, lr=lr, beta1=beta1, beta2=beta2, eps=eps, gemm_mode=gemm_mode,
                      agg_mode=agg_mode, loss_rows_only=loss_rows_only, epoch_graph=epoch_graph,
                      factored_norm=factored_norm, cache_ax=cache_ax)
        for i, d in enumerate(dims[:MAX_LAYERS + 1]):
            o.dims[i] = int(d)
        ws = [_np(w, np.float32) for w in w0]
        bs = [None if b is None else _np(b, np.float32) for b in (list(b0) if b0 is not None else [None] * L)]
        wp = (C.c_void_p * max(L, 1))(*[w.ctypes.data for w in ws])
        bp = (C.c_void_p * max(L, 1))(*[None if b is None else b.ctypes.data for b in bs])
        self.env, self.parts, self.dims, self.L = env, parts, list(dims), L
        self.handle = C.c_void_p()
        _ck(lib().gcnsa_model_create(C.byref(env), parts.handle, C.byref(o), wp, bp, C.byref(self.handle)))

    def forward(self, p, loss_dev_ptr=None):
        _ck(lib().gcnsa_forward(self.handle, self.parts.handle, p, loss_dev_ptr))

    def backward(self, p):
        _ck(lib().gcnsa_backward(self.handle, self.parts.handle, p))

    def step(self):
        _ck(lib().gcnsa_step(self.handle))

    def epoch(self, loss_dev_ptr=None):
        _ck(lib().gcnsa_epoch(self.handle, self.parts.handle, loss_dev_ptr))

    def epoch_host(self, x_host_ptrs, loss_host: np.ndarray):
        arr = (C.c_void_p * len(x_host_ptrs))(*x_host_ptrs)
        _ck(lib().gcnsa_epoch_host(self.handle, self.parts.handle, arr, _hp(loss_host)))

    def get(self, what, layer=0, rows=None) -> np.ndarray:
        if what in (GET_ACT, GET_DLOGITS):
            cols = self.dims[layer] if what == GET_ACT else self.dims[-1]
            out = np.empty((rows, cols), np.float32)
        elif what in (GET_W, GET_GRAD_W, GET_ADAM_M_W, GET_ADAM_V_W):
            out = np.empty((self.dims[layer], self.dims[layer + 1]), np.float32)
        else:
            out = np.empty(self.dims[layer + 1], np.float32)
        _ck(lib().gcnsa_model_get(self.handle, what, layer, _hp(out), out.nbytes))
        return out

    def set(self, what, layer, value):
        v = _np(value, np.float32)
        _ck(lib().gcnsa_model_set(self.handle, what, layer, _hp(v), v.nbytes))

    def evaluate(self, parts, p=0, mask=None):
        """(correct, total, predictions) of the current parameters on partition p of `parts`;
        micro-F1 (= accuracy) is correct / total."""
        n = parts.info(p).n
        pred = np.empty(n, np.int32)
        mk = None if mask is None else _np(mask, np.uint8)
        correct, total = C.c_int64(), C.c_int64()
        _ck(lib().gcnsa_evaluate(self.handle, parts.handle, p, _hp(mk), C.byref(correct), C.byref(total), _hp(pred)))
        return int(correct.value), int(total.value), pred

    def copy_params_from(self, other):
        _ck(lib().gcnsa_model_copy_params(self.handle, other.handle))

    def select_partition(self, p):
        """Whose Adam moments get / set address when every partition has its own (AGG_PARAM_AVG)."""
        _ck(lib().gcnsa_model_select_partition(self.handle, p))

    def profile(self, enable: bool):
        _ck(lib().gcnsa_model_profile(self.handle, 1 if enable else 0))

    def profile_read(self) -> dict:
        pr = Profile()
        _ck(lib().gcnsa_model_profile_read(self.handle, C.byref(pr)))
        names = ("spmm", "gemm", "other")
        return {nm: {"ms": pr.ms[i], "launches": int(pr.launches[i]), "alg_bytes": pr.alg_bytes[i], "flops": pr.flops[i],
                     "l1_bytes": pr.l1_bytes[i], "alg_bytes_val": pr.alg_bytes_val[i]} for i, nm in enumerate(names)}

    @property
    def t(self) -> int:
        out = C.c_int64()
        _ck(lib().gcnsa_model_get_t(self.handle, C.byref(out)))
        return int(out.value)

    @t.setter
    def t(self, value):
        _ck(lib().gcnsa_model_set_t(self.handle, int(value)))

    def close(self):
        if self.handle:
            lib().gcnsa_model_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:  # noqa: BLE001
            pass


(SAGE_W_SELF, SAGE_W_NEIGH, SAGE_B, SAGE_WORK_W_SELF, SAGE_WORK_W_NEIGH, SAGE_WORK_B, SAGE_GRAD_W_SELF, SAGE_GRAD_W_NEIGH,
 SAGE_GRAD_B) = range(9)


class Sage:
    """GraphSAGE with the mean aggregator on one set of partitions: two layers, per-worker copies of the
    parameters with their own Adam state, averaged once per epoch."""

    def __init__(self, env: Env, parts: Parts, dims, w_self0, w_neigh0, b0=None, fanout=(25, 10), batch=256, lr=1e-4,
                 beta1=0.9, beta2=0.999, eps=1e-8, seed=0, gemm_mode=GEMM_TF32X3, batch_graph=1):
        assert len(dims) == 3 and len(fanout) == 2
        o = SageOpts(batch=batch, lr=lr, beta1=beta1, beta2=beta2, eps=eps, seed=seed, gemm_mode=gemm_mode,
                     batch_graph=batch_graph)
        for i, d in enumerate(dims):
            o.dims[i] = int(d)
        o.fanout[0], o.fanout[1] = int(fanout[0]), int(fanout[1])
        ws = [_np(w, np.float32) for w in w_self0]
        wn = [_np(w, np.float32) for w in w_neigh0]
        bs = [None if b is None else _np(b, np.float32) for b in (list(b0) if b0 is not None else [None, None])]
        mk = lambda arrs: (C.c_void_p * 2)(*[None if a is None else a.ctypes.data for a in arrs])  # noqa: E731
        self.env, self.parts, self.dims, self.fanout, self.batch = env, parts, list(dims), tuple(fanout), batch
        self.handle = C.c_void_p()
        _ck(lib().gcnsa_sage_create(C.byref(env), parts.handle, C.byref(o), mk(ws), mk(wn), mk(bs), C.byref(self.handle)))

    def epoch(self, loss_dev_ptr=None):
        _ck(lib().gcnsa_sage_epoch(self.handle, self.parts.handle, loss_dev_ptr))

    @property
    def epochs_done(self) -> int:
        out = C.c_int64()
        _ck(lib().gcnsa_sage_get_epoch(self.handle, C.byref(out)))
        return int(out.value)

    def profile(self, enable: bool):
        _ck(lib().gcnsa_sage_profile(self.handle, 1 if enable else 0))

    def profile_read(self) -> dict:
        pr = Profile()
        _ck(lib().gcnsa_sage_profile_read(self.handle, C.byref(pr)))
        names = ("gather", "gemm", "other")
        return {nm: {"ms": pr.ms[i], "launches": int(pr.launches[i]), "alg_bytes": pr.alg_bytes[i], "flops": pr.flops[i]}
                for i, nm in enumerate(names)}

    def n_batches(self, p) -> int:
        out = C.c_int64()
        _ck(lib().gcnsa_sage_batches(self.handle, self.parts.handle, p, C.byref(out)))
        return int(out.value)

    def run_batch(self, p, epoch, b, apply=False, loss_dev_ptr=None):
        _ck(lib().gcnsa_sage_batch(self.handle, self.parts.handle, p, epoch, b, 1 if apply else 0, loss_dev_ptr))

    def batch_export(self) -> dict:
        nb, rows1 = C.c_int64(), C.c_int64()
        _ck(lib().gcnsa_sage_batch_shape(self.handle, C.byref(nb), C.byref(rows1)))
        nb, rows1 = int(nb.value), int(rows1.value)
        out = {"vertices": np.empty(rows1, np.int32), "count2": np.empty(nb, np.int32),
               "samples1": np.empty((rows1, self.fanout[0]), np.int32), "count1": np.empty(rows1, np.int32),
               "hidden": np.empty((rows1, self.dims[1]), np.float32), "logits": np.empty((nb, self.dims[2]), np.float32),
               "dlogits": np.empty((nb, self.dims[2]), np.float32), "loss": np.empty(1, np.float32)}
        h = SageBatchHost(**{k: _hp(v) for k, v in out.items()})
        _ck(lib().gcnsa_sage_batch_export(self.handle, C.byref(h)))
        out["nb"] = nb
        return out

    def get(self, what, layer) -> np.ndarray:
        ok = 0 <= layer <= 1     # the library reports a bad layer or tensor id; only the buffer is sized here
        din, dout = (self.dims[layer], self.dims[layer + 1]) if ok else (1, 1)
        out = np.empty(dout if what % 3 == 2 else (din, dout), np.float32)
        _ck(lib().gcnsa_sage_get(self.handle, what, layer, _hp(out), out.nbytes))
        return out

    def close(self):
        if self.handle:
            lib().gcnsa_sage_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:  # noqa: BLE001
            pass


# ------------------------------------------------- single ops on torch tensors ---
def _dp(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def op_spmm(rowptr, col, val, x, f, y, epi=EPI_NONE, aux=None, order=None, n_long=0):
    ldaux = 0 if aux is None or aux.dim() == 1 else aux.stride(0)
    _ck(lib().gcnsa_op_spmm(_stream(), rowptr.numel() - 1, _dp(rowptr), _dp(col), _dp(val), _dp(order), n_long, _dp(x),
                            x.stride(0), f, epi, _dp(aux), ldaux, _dp(y), y.stride(0)))


def op_spmm_pattern(rowptr, col, x, f, y, row_scale=None, epi=EPI_NONE, aux=None, order=None, n_long=0):
    """Y = epi(diag(row_scale) B X) with B the 0/1 pattern of the CSR (no values read)."""
    ldaux = 0 if aux is None or aux.dim() == 1 else aux.stride(0)
    _ck(lib().gcnsa_op_spmm_pattern(_stream(), rowptr.numel() - 1, _dp(rowptr), _dp(col), _dp(row_scale), _dp(order),
                                    n_long, _dp(x), x.stride(0), f, epi, _dp(aux), ldaux, _dp(y), y.stride(0)))


def op_gemm(a, b, c, m, n, k, ta=0, tb=0, accumulate=0, epi=EPI_NONE, aux=None, workspace=None, mode=GEMM_FP32):
    ldaux = 0 if aux is None or aux.dim() == 1 else aux.stride(0)
    wb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _ck(lib().gcnsa_op_gemm(_stream(), mode, ta, tb, m, n, k, _dp(a), a.stride(0), _dp(b), b.stride(0), _dp(c),
                            c.stride(0), accumulate, epi, _dp(aux), ldaux, _dp(workspace), wb))


def op_gemm_workspace(ta, tb, m, n, k, mode=GEMM_FP32) -> int:
    return int(lib().gcnsa_op_gemm_workspace(mode, ta, tb, m, n, k))


def op_gemm_mask_colsum(a, b, c, m, n, k, mask, out, row_scale=None, ta=0, tb=0, accumulate=0, scratch=None,
                        workspace=None, mode=GEMM_FP32):
    sb = 0 if scratch is None else scratch.numel() * scratch.element_size()
    wb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _ck(lib().gcnsa_op_gemm_mask_colsum(_stream(), mode, ta, tb, m, n, k, _dp(a), a.stride(0), _dp(b), b.stride(0), _dp(c),
                                        c.stride(0), _dp(mask), mask.stride(0), _dp(row_scale), _dp(out), accumulate,
                                        _dp(scratch), sb, _dp(workspace), wb))


def op_gemm_mask_colsum_scratch(m, n) -> int:
    return int(lib().gcnsa_op_gemm_mask_colsum_scratch(m, n))


def gather_probe_warps() -> int:
    out = C.c_int32()
    _ck(lib().gcnsa_op_gather_probe_warps(C.byref(out)))
    return int(out.value)


def op_gather_probe(x, n_rows, window_rows, hit_every, rounds, out):
    """Gathers rounds x 16 rows of 512 bytes per warp (see include/gcnsa.h); out: float32 [warps x 128]."""
    _ck(lib().gcnsa_op_gather_probe(_stream(), _dp(x), x.stride(0), n_rows, window_rows, hit_every, rounds, _dp(out),
                                    out.numel() * out.element_size()))


def debug_status() -> tuple:
    """(enabled, code, value) of the checking build's record; enabled is False for the regular library."""
    en, code, val = C.c_int32(), C.c_int32(), C.c_int64()
    _ck(lib().gcnsa_debug_status(C.byref(en), C.byref(code), C.byref(val)))
    return bool(en.value), int(code.value), int(val.value)


def use_library(path: str):
    """Load another build of the library (the checking build) instead of the default one; before the first call."""
    global LIB_PATH
    if _lib is not None:
        raise RuntimeError("the library is loaded already")
    LIB_PATH = path


def tc_clear():
    """Resets the error word of the tensor-core kernels."""
    _ck(lib().gcnsa_tc_clear())


def tc_status() -> int:
    """Error word of the tensor-core kernels after a device synchronize (0 = healthy)."""
    out = C.c_int32()
    _ck(lib().gcnsa_tc_status(C.byref(out)))
    return int(out.value)


def op_softmax_ce(logits, c, y, mask, n_train, loss, grad, scratch):
    _ck(lib().gcnsa_op_softmax_ce(_stream(), logits.shape[0], c, _dp(logits), logits.stride(0), _dp(y), _dp(mask),
                                  n_train, _dp(loss), _dp(grad), grad.stride(0), _dp(scratch),
                                  scratch.numel() * scratch.element_size()))


def op_softmax_ce_scratch(n) -> int:
    return int(lib().gcnsa_op_softmax_ce_scratch(n))


def op_colsum(g, f, out, accumulate, scratch):
    _ck(lib().gcnsa_op_colsum(_stream(), g.shape[0], f, _dp(g), g.stride(0), _dp(out), accumulate, _dp(scratch),
                              scratch.numel() * scratch.element_size()))


def op_colsum_scaled(g, f, out, accumulate, scratch, row_scale, scaled):
    """Column sums of g and, in the same pass, scaled = diag(row_scale) g (scaled may be g)."""
    _ck(lib().gcnsa_op_colsum_scaled(_stream(), g.shape[0], f, _dp(g), g.stride(0), _dp(out), accumulate, _dp(scratch),
                                     scratch.numel() * scratch.element_size(), _dp(row_scale), _dp(scaled),
                                     scaled.stride(0)))


def op_colsum_static(g, f, out, accumulate):
    """Column sums with the library's built-in scratch: allocates nothing (for
    callers that may not call cudaMalloc); f is limited to COLSUM_STATIC_MAX_F."""
    _ck(lib().gcnsa_op_colsum_static(_stream(), g.shape[0], f, _dp(g), g.stride(0), _dp(out), accumulate))


COLSUM_STATIC_MAX_F = 1024


def op_colsum_scratch(n, f) -> int:
    return int(lib().gcnsa_op_colsum_scratch(n, f))


def op_adam(theta, gsum, m, v, inv_m, lr, beta1, beta2, eps, t):
    _ck(lib().gcnsa_op_adam(_stream(), theta.numel(), _dp(theta), _dp(gsum), _dp(m), _dp(v), inv_m, lr, beta1, beta2,
                            eps, t))


def op_normalize(rowptr, col, deg, val):
    _ck(lib().gcnsa_op_normalize(_stream(), rowptr.numel() - 1, _dp(rowptr), _dp(col), _dp(deg), _dp(val)))
