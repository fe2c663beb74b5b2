"""ctypes binding of ``libgcn_admm.so``: argument marshalling only.

Every function of ``include/gcn_admm.h`` has a counterpart of the same name on ``GcnAdmm``
(without the ``gcn_admm_`` prefix).  Nothing is computed here; the library must have been built
(``python -m paper_2112_09335_b200.build``) or loading fails with an error -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libgcn_admm.so")

EXPORTS = [
    "gcn_admm_default_params", "gcn_admm_create", "gcn_admm_step", "gcn_admm_objective", "gcn_admm_weights",
    "gcn_admm_predict", "gcn_admm_destroy", "gcn_admm_last_error", "gcn_admm_propagate", "gcn_admm_index",
    "gcn_admm_get_state", "gcn_admm_set_state", "gcn_admm_step_block", "gcn_admm_decisions",
    "gcn_admm_launches", "gcn_admm_profile", "gcn_admm_profile_read", "gcn_admm_propagate_static", "gcn_admm_dense_product", "gcn_admm_dense_product_tn",
    "gcn_admm_shard_plan", "gcn_admm_propagate_sharded",
]

IX = dict(perm=0, inv_perm=1, comm_ptr=2, nbr=3, halo1=4, halo2=5, csr_row_ptr=6, csr_col=7,
          seg_row_ptr=8, seg_comm=9, seg_begin=10)
ST_W, ST_Z, ST_U, ST_TAU, ST_THETA, ST_PIPELINE_FLAG = range(6)
PHASE_W, PHASE_Z, PHASE_U = range(3)


class Params(C.Structure):
    _fields_ = [("nu", C.c_float), ("rho", C.c_float), ("tau0", C.c_float), ("theta0", C.c_float),
                ("bt_growth", C.c_float), ("bt_shrink", C.c_float), ("bt_max_trials", C.c_int),
                ("fista_iters", C.c_int), ("loss_scale", C.c_float), ("dual_mode", C.c_int), ("tensor_cores", C.c_int), ("use_graph", C.c_int), ("schedule", C.c_int), ("long_row", C.c_int),
                ("seed", C.c_ulonglong), ("w_init", C.POINTER(C.POINTER(C.c_float))), ("device", C.c_int), ("stream", C.c_void_p)]


class GcnAdmmError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"gcn_admm error {code}: {msg}")
        self.code = code


_lib = None


def load():
    """Loads the shared library (once) and declares the signatures."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2112_09335_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int, C.c_longlong
    lib.gcn_admm_default_params.argtypes = [C.POINTER(Params)]
    lib.gcn_admm_default_params.restype = None
    lib.gcn_admm_create.argtypes = [C.POINTER(vp), i64, vp, vp, vp, vp, vp, i32, C.POINTER(i32), C.POINTER(Params),
                                    i32, vp]
    lib.gcn_admm_step.argtypes = [vp, i32]
    lib.gcn_admm_objective.argtypes = [vp, C.POINTER(C.c_double)]
    lib.gcn_admm_weights.argtypes = [vp, i32, vp]
    lib.gcn_admm_predict.argtypes = [vp, vp, vp]
    lib.gcn_admm_destroy.argtypes = [vp]
    lib.gcn_admm_destroy.restype = None
    lib.gcn_admm_last_error.argtypes = [vp]
    lib.gcn_admm_last_error.restype = C.c_char_p
    lib.gcn_admm_propagate.argtypes = [vp, vp, i32, vp]
    lib.gcn_admm_propagate_static.argtypes = [vp, vp, i32, vp]
    lib.gcn_admm_propagate_sharded.argtypes = [vp, i32, vp, i32, vp, C.POINTER(i64)]
    lib.gcn_admm_dense_product.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32]
    lib.gcn_admm_dense_product_tn.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32]
    lib.gcn_admm_index.argtypes = [vp, i32, i32, C.POINTER(C.POINTER(i32)), C.POINTER(i64)]
    lib.gcn_admm_shard_plan.argtypes = [vp, i32, i32, i32, i32, C.POINTER(C.POINTER(i32)), C.POINTER(i64)]
    lib.gcn_admm_get_state.argtypes = [vp, i32, i32, vp]
    lib.gcn_admm_set_state.argtypes = [vp, i32, i32, vp]
    lib.gcn_admm_step_block.argtypes = [vp, i32, i32]
    lib.gcn_admm_decisions.argtypes = [vp, i32, C.POINTER(i32), vp, vp, vp, vp]
    lib.gcn_admm_launches.argtypes = [vp, C.POINTER(i64)]
    lib.gcn_admm_profile.argtypes = [vp, i32]
    lib.gcn_admm_profile_read.argtypes = [vp, i32, C.POINTER(i32), vp, vp, vp, vp, vp]
    _lib = lib
    return lib


def _ptr(a):
    """Address of a numpy array, or the raw value of an int (a device pointer)."""
    if a is None:
        return None
    if isinstance(a, int):
        return C.c_void_p(a)
    return a.ctypes.data_as(C.c_void_p)


def default_params() -> Params:
    p = Params()
    load().gcn_admm_default_params(C.byref(p))
    return p


class GcnAdmm:
    """Owner of one library handle.  Array arguments are numpy arrays (host) or, for ``create``'s
    graph / feature inputs and ``propagate``, integers holding device addresses."""

    def __init__(self, n, row_ptr, col_idx, X, y, train_mask, widths, n_comm, community, w_init, nu=1e-3, rho=1e-3,
                 tau0=1.0, theta0=1.0, bt_growth=2.0, bt_shrink=0.5, bt_max_trials=40, fista_iters=30,
                 loss_scale=1.0, dual_mode=0, tensor_cores=1, use_graph=2, schedule=0, long_row=0, seed=0, device=0, stream=0):
        lib = load()
        self._lib = lib
        self._h = C.c_void_p()
        self.n, self.widths, self.n_comm = int(n), [int(w) for w in widths], int(n_comm)
        self.L = len(self.widths) - 1
        p = default_params()
        p.nu, p.rho, p.tau0, p.theta0 = nu, rho, tau0, theta0
        p.bt_growth, p.bt_shrink, p.bt_max_trials = bt_growth, bt_shrink, bt_max_trials
        p.fista_iters, p.loss_scale, p.dual_mode = fista_iters, loss_scale, dual_mode
        p.tensor_cores = int(tensor_cores)
        p.use_graph = int(use_graph)
        p.schedule = int(schedule)
        p.long_row = int(long_row)
        p.seed = int(seed)
        p.device, p.stream = device, stream or None
        if w_init is not None:
            ws = [np.ascontiguousarray(w, dtype=np.float32) for w in w_init]
            arr = (C.POINTER(C.c_float) * len(ws))(*[w.ctypes.data_as(C.POINTER(C.c_float)) for w in ws])
            p.w_init = C.cast(arr, C.POINTER(C.POINTER(C.c_float)))
        keep = []

        def host(a, dt):
            if isinstance(a, int):
                return a
            b = np.ascontiguousarray(a, dtype=dt)
            keep.append(b)
            return b
        wd = (C.c_int * len(self.widths))(*self.widths)
        rc = lib.gcn_admm_create(C.byref(self._h), self.n, _ptr(host(row_ptr, np.int64)), _ptr(host(col_idx, np.int32)),
                                 _ptr(host(X, np.float32)), _ptr(host(y, np.int32)),
                                 _ptr(host(train_mask, np.uint8)), self.L, wd, C.byref(p), self.n_comm,
                                 _ptr(host(community, np.int32)))
        if rc != 0:
            raise GcnAdmmError(rc, lib.gcn_admm_last_error(None).decode())

    def _check(self, rc):
        if rc != 0:
            raise GcnAdmmError(rc, self._lib.gcn_admm_last_error(self._h).decode())

    def destroy(self):
        if getattr(self, "_h", None) and self._h.value:
            self._lib.gcn_admm_destroy(self._h)
            self._h = C.c_void_p()

    __del__ = destroy

    def step(self, n_iters=1):
        self._check(self._lib.gcn_admm_step(self._h, int(n_iters)))

    def step_block(self, phase, layer=0):
        self._check(self._lib.gcn_admm_step_block(self._h, int(phase), int(layer)))

    def objective(self):
        out = (C.c_double * 6)()
        self._check(self._lib.gcn_admm_objective(self._h, out))
        return np.array(out[:])

    def weights(self, layer):
        shape = (self.widths[layer - 1], self.widths[layer]) if 1 <= layer <= self.L else (1, 1)   # the library rejects it
        out = np.empty(shape, dtype=np.float32)
        self._check(self._lib.gcn_admm_weights(self._h, layer, _ptr(out)))
        return out

    def predict(self):
        logits = np.empty((self.n, self.widths[-1]), dtype=np.float32)
        labels = np.empty(self.n, dtype=np.int32)
        self._check(self._lib.gcn_admm_predict(self._h, _ptr(logits), _ptr(labels)))
        return logits, labels

    def propagate(self, x, width=None, out=None):
        """A~ x.  numpy in -> numpy out; device addresses (ints) in -> ``out`` must be given."""
        if isinstance(x, int):
            self._check(self._lib.gcn_admm_propagate(self._h, _ptr(x), int(width), _ptr(out)))
            return out
        x = np.ascontiguousarray(x, dtype=np.float32)
        res = np.empty_like(x)
        self._check(self._lib.gcn_admm_propagate(self._h, _ptr(x), x.shape[1], _ptr(res)))
        return res

    def propagate_static(self, x_dev, width, out_dev):
        """A~ x between device buffers (addresses as ints) using the library's built-in staging
        memory: nothing is allocated by the call.  Enqueued on the handle's stream."""
        self._check(self._lib.gcn_admm_propagate_static(self._h, _ptr(int(x_dev)), int(width), _ptr(int(out_dev))))

    def dense_product(self, a_dev, b_dev, c_dev, m, n, k, tensor_cores=1):
        """C = A B between dense device buffers (addresses as ints)."""
        self._check(self._lib.gcn_admm_dense_product(self._h, _ptr(int(a_dev)), _ptr(int(b_dev)), _ptr(int(c_dev)), int(m),
                                                     int(n), int(k), int(tensor_cores)))

    def dense_product_tn(self, a_dev, b_dev, c_dev, rows, ka, nb, tensor_cores=1):
        """C = A^T B between dense device buffers (addresses as ints): A rows x ka, B rows x nb."""
        self._check(self._lib.gcn_admm_dense_product_tn(self._h, _ptr(int(a_dev)), _ptr(int(b_dev)), _ptr(int(c_dev)),
                                                        int(rows), int(ka), int(nb), int(tensor_cores)))

    def index(self, which, comm=0):
        data = C.POINTER(C.c_int)()
        length = C.c_longlong()
        self._check(self._lib.gcn_admm_index(self._h, IX[which], int(comm), C.byref(data), C.byref(length)))
        if length.value == 0:
            return np.zeros(0, dtype=np.int32)
        return np.ctypeslib.as_array(data, shape=(length.value,)).copy()

    def shard_plan(self, n_ranks, which, receiver=0, sender=0):
        """which: 0 ranges (first community / row of every rank, concatenated), 1 first-order rows, 2 second-order rows."""
        data = C.POINTER(C.c_int)()
        length = C.c_longlong()
        self._check(self._lib.gcn_admm_shard_plan(self._h, int(n_ranks), int(which), int(receiver), int(sender),
                                                  C.byref(data), C.byref(length)))
        if length.value == 0:
            return np.zeros(0, dtype=np.int32)
        return np.ctypeslib.as_array(data, shape=(length.value,)).copy()

    def propagate_sharded(self, n_ranks, x):
        """A~ x formed rank by rank from each rank's own rows and copies of its first-order rows (numpy in,
        numpy out); also returns the number of first-order rows copied, summed over the ranks."""
        x = np.ascontiguousarray(x, dtype=np.float32)
        res = np.empty_like(x)
        staged = C.c_longlong()
        self._check(self._lib.gcn_admm_propagate_sharded(self._h, int(n_ranks), _ptr(x), x.shape[1], _ptr(res),
                                                         C.byref(staged)))
        return res, staged.value

    def _state_shape(self, which, layer):
        if which in (ST_W, ST_Z) and not 1 <= layer <= self.L:
            return (1,), np.float32            # out of range: left to the library to reject
        if which == ST_W:
            return (self.widths[layer - 1], self.widths[layer]), np.float32
        if which == ST_Z:
            return (self.n, self.widths[layer]), np.float32
        if which == ST_U:
            return (self.n, self.widths[-1]), np.float32
        if which == ST_TAU:
            return (1,), np.float64
        if which == ST_PIPELINE_FLAG:
            return (1,), np.int32
        return (self.n_comm,), np.float64

    def get_state(self, which, layer=0):
        shape, dt = self._state_shape(which, layer)
        out = np.empty(shape, dtype=dt)
        self._check(self._lib.gcn_admm_get_state(self._h, which, layer, _ptr(out)))
        return out

    def set_state(self, which, layer, value):
        shape, dt = self._state_shape(which, layer)
        v = np.ascontiguousarray(value, dtype=dt).reshape(shape)
        self._check(self._lib.gcn_admm_set_state(self._h, which, layer, _ptr(v)))

    def launches(self):
        c = C.c_longlong()
        self._check(self._lib.gcn_admm_launches(self._h, C.byref(c)))
        return c.value

    def profile(self, enable):
        self._check(self._lib.gcn_admm_profile(self._h, 1 if enable else 0))

    def profile_read(self, max_entries=128):
        n = C.c_int()
        names = C.create_string_buffer(max_entries * 48)
        la = np.zeros(max_entries, dtype=np.int64)
        ms, by, fl = (np.zeros(max_entries) for _ in range(3))
        self._check(self._lib.gcn_admm_profile_read(self._h, max_entries, C.byref(n), names, _ptr(la), _ptr(ms), _ptr(by),
                                                    _ptr(fl)))
        out = {}
        for k in range(n.value):
            name = names.raw[k * 48:(k + 1) * 48].split(b"\0")[0].decode()
            out[name] = dict(launches=int(la[k]), ms=float(ms[k]), bytes=float(by[k]), flops=float(fl[k]))
        return out

    def decisions(self, max_passes=256):
        L, M = self.L, self.n_comm
        n = C.c_int()
        tw = np.empty((max_passes, L), dtype=np.int32)
        qw = np.empty((max_passes, L), dtype=np.float64)
        tz = np.empty((max_passes, max(L - 1, 0), M), dtype=np.int32)
        qz = np.empty((max_passes, max(L - 1, 0), M), dtype=np.float64)
        self._check(self._lib.gcn_admm_decisions(self._h, max_passes, C.byref(n), _ptr(tw), _ptr(qw), _ptr(tz), _ptr(qz)))
        k = n.value
        return dict(trial_w=tw[:k], q_w=qw[:k], trial_z=tz[:k], q_z=qz[:k])
