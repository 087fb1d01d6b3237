"""ctypes loader for the CodeNet CPU oracle -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It compiles ``codenet_oracle.c`` with gcc on first use and exposes thin numpy wrappers.  It
imports nothing from the CUDA package.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "codenet_oracle.c")
_HDR = os.path.join(_HERE, "codenet_oracle.h")
_LIB = os.path.join(_HERE, "libcodenet_oracle.so")

LOCATE_NONE, LOCATE_SYNDROME, LOCATE_NODECHECK = 0, 1, 2
LOCATE_JOINT = 4
FAULT_NONE, FAULT_BERNOULLI, FAULT_EXACTLY_ONE = 0, 1, 2
PHASE_FWD, PHASE_BWD = 0, 1
CLEAN, CORRECTED, FALLBACK, FAILED = 0, 1, 2, 3
ACT_IDENTITY, ACT_RELU = 0, 1
LOSS_MSE_MEAN, LOSS_SOFTMAX_CE = 0, 1


def build(force=False):
    """Compile the oracle shared library (gcc -O2, OpenMP)."""
    if not force and os.path.exists(_LIB):
        newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
        if os.path.getmtime(_LIB) >= newest:
            return _LIB
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


class Desc(C.Structure):
    _fields_ = [("n_out", C.c_int32), ("n_in", C.c_int32), ("m", C.c_int32), ("n", C.c_int32),
                ("r_row", C.c_int32), ("r_col", C.c_int32), ("store_bf16", C.c_int32),
                ("locate_mode", C.c_int32), ("check_rows", C.c_int32), ("check_cols", C.c_int32),
                ("tau_rel", C.c_float), ("tau_abs", C.c_float),
                ("P_row", C.POINTER(C.c_float)), ("P_col", C.POINTER(C.c_float))]


class Fault(C.Structure):
    _fields_ = [("seed", C.c_uint32), ("layer", C.c_uint32), ("mode", C.c_uint32),
                ("p_q32", C.c_uint32), ("sigma", C.c_float)]


class SmallFaults(C.Structure):
    _fields_ = [("seed", C.c_uint32), ("layer", C.c_uint32), ("p_encode_q32", C.c_uint32), ("p_input_q32", C.c_uint32),
                ("p_check_q32", C.c_uint32), ("p_decode_q32", C.c_uint32), ("sigma", C.c_float)]


class Report(C.Structure):
    _fields_ = [("status", C.c_uint32), ("n_detected_cw", C.c_uint32),
                ("n_flagged_nodes", C.c_uint32), ("n_fallback_cw", C.c_uint32),
                ("detected_mask", C.c_uint64), ("flagged_mask", C.c_uint64 * 64),
                ("injected_mask", C.c_uint64 * 64),
                ("min_margin_hit", C.c_float), ("max_margin_clean", C.c_float)]

    def decisions(self):
        """The integer part of the report: what must agree bit for bit."""
        return (int(self.status), int(self.n_detected_cw), int(self.n_flagged_nodes),
                int(self.n_fallback_cw), int(self.detected_mask),
                tuple(int(x) for x in self.flagged_mask), tuple(int(x) for x in self.injected_mask))


_lib = None


def lib():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(build())
    fp = C.POINTER(C.c_float)
    vp = C.c_void_p
    L.orc_set_threads.argtypes = [C.c_int]
    L.orc_get_threads.restype = C.c_int
    L.orc_philox4x32_10.argtypes = [C.POINTER(C.c_uint32)] * 3
    L.orc_noise.argtypes = [C.c_uint32] * 6 + [C.c_float]
    L.orc_noise.restype = C.c_float
    L.orc_node_hit.argtypes = [C.POINTER(Fault)] + [C.c_uint32] * 5
    L.orc_node_hit.restype = C.c_int
    L.orc_layer_create.argtypes = [C.POINTER(Desc), fp]
    L.orc_layer_create.restype = vp
    L.orc_layer_free.argtypes = [vp]
    L.orc_layer_dims.argtypes = [vp, C.POINTER(C.c_int32)]
    for name in ("orc_get_block", "orc_get_u", "orc_get_v", "orc_set_block"):
        getattr(L, name).argtypes = [vp, C.c_int, C.c_int, fp]
        getattr(L, name).restype = C.c_int
    L.orc_corrupt_block.argtypes = [vp, C.c_int, C.c_int, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, C.c_float]
    L.orc_corrupt_block.restype = C.c_long
    L.orc_regenerate_block.argtypes = [vp, C.c_int, C.c_int, C.c_int]
    L.orc_regenerate_block.restype = C.c_int
    L.orc_checkpoint_save.argtypes = [vp]
    L.orc_checkpoint_save.restype = C.c_int
    L.orc_checkpoint_restore.argtypes = [vp]
    L.orc_checkpoint_restore.restype = C.c_int
    L.orc_encode_x.argtypes = [vp, fp, C.c_int, fp]
    L.orc_encode_delta.argtypes = [vp, fp, C.c_int, fp]
    L.orc_forward_products.argtypes = [vp, fp, C.c_int, fp]
    L.orc_backward_products.argtypes = [vp, fp, C.c_int, fp]
    L.orc_inject.argtypes = [vp, C.c_int, C.POINTER(Fault), C.c_uint32, fp, C.c_int,
                             C.POINTER(C.c_uint64)]
    L.orc_detect_decode.argtypes = [vp, C.c_int, fp, fp, C.c_int, fp, C.POINTER(C.c_uint64),
                                    C.POINTER(Report)]
    L.orc_forward.argtypes = [vp, fp, C.c_int, C.POINTER(Fault), C.c_uint32, fp, C.POINTER(Report)]
    L.orc_update.argtypes = [vp, fp, fp, C.c_int, C.c_float]
    L.orc_backward_update.argtypes = [vp, fp, fp, C.c_int, C.c_float, C.POINTER(Fault),
                                      C.c_uint32, fp, C.POINTER(Report)]
    L.orc_decode_weights.argtypes = [vp, fp]
    L.orc_layer_set_small_faults.argtypes = [vp, C.POINTER(SmallFaults)]
    L.orc_layer_set_small_faults.restype = None
    L.orc_small_hit.argtypes = [C.POINTER(SmallFaults), C.c_uint32, C.c_uint32, C.c_uint32]
    L.orc_small_hit.restype = C.c_int
    L.orc_code_conditioning.argtypes = [vp, C.c_int, C.POINTER(C.c_double)]
    L.orc_code_conditioning.restype = None
    L.orc_check_invariance.argtypes = [vp]
    L.orc_check_invariance.restype = C.c_double
    L.orc_net_create.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int]
    L.orc_net_create.restype = vp
    L.orc_net_free.argtypes = [vp]
    L.orc_step.argtypes = [vp, fp, vp, C.c_int, C.c_float, C.POINTER(Fault), C.c_uint32,
                           C.POINTER(Report), fp, fp]
    _lib = L
    return L


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _fp(a):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def set_threads(n):
    lib().orc_set_threads(int(n))


def get_threads():
    return int(lib().orc_get_threads())


def philox(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def noise(seed, layer, phase, iteration, node_id, element, sigma):
    return float(lib().orc_noise(seed, layer, phase, iteration, node_id, element, sigma))


def make_fault(seed=0, layer=0, mode=FAULT_NONE, p=0.0, sigma=10.0):
    p_q32 = min(int(p * 4294967296.0), 0xFFFFFFFF)
    return Fault(seed, layer, mode, p_q32, sigma)


DISAGREE = 5
PHASE_ENCODE, PHASE_INPUT, PHASE_CHECK, PHASE_DECODE = 2, 3, 4, 5


def make_small_faults(seed=0, layer=0, p_encode=0.0, p_input=0.0, p_check=0.0, p_decode=0.0, sigma=10.0):
    q = lambda p: min(int(p * 4294967296.0), 0xFFFFFFFF)
    return SmallFaults(seed, layer, q(p_encode), q(p_input), q(p_check), q(p_decode), sigma)


def small_hit(plan, phase, iteration, unit):
    return bool(lib().orc_small_hit(C.byref(plan), phase, iteration, unit))


def node_hit(fault, phase, iteration, node_id, active_index, n_active):
    return bool(lib().orc_node_hit(C.byref(fault), phase, iteration, node_id, active_index, n_active))


class Layer:
    """One coded layer held by the oracle."""

    def __init__(self, W, m, n, r_row, r_col, P_row=None, P_col=None, store_bf16=False,
                 locate_mode=LOCATE_NODECHECK, check_rows=0, check_cols=0, tau_rel=1e-3, tau_abs=1e-20):
        W = _f32(W)
        self.n_out, self.n_in = W.shape
        self._P_row = None if P_row is None else _f32(P_row).reshape(m, r_row)
        self._P_col = None if P_col is None else _f32(P_col).reshape(n, r_col)
        d = Desc(self.n_out, self.n_in, m, n, r_row, r_col, int(store_bf16), locate_mode,
                 check_rows, check_cols, tau_rel, tau_abs,
                 None if self._P_row is None else _fp(self._P_row),
                 None if self._P_col is None else _fp(self._P_col))
        self.h = lib().orc_layer_create(C.byref(d), _fp(W))
        if not self.h:
            raise ValueError("oracle rejected the layer description")
        dims = (C.c_int32 * 10)()
        lib().orc_layer_dims(self.h, dims)
        (self.b_r, self.b_c, self.M, self.Nn, self.T, self.ns, self.n_out_p, self.n_in_p, self.Tc,
         self.nsc) = [int(x) for x in dims]
        self.m, self.n, self.r_row, self.r_col = m, n, r_row, r_col

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_layer_free(self.h)
            self.h = None

    def has_node(self, i, j):
        return i < self.M and j < self.Nn and (i < self.m or j < self.n)

    def block(self, i, j):
        out = np.empty((self.b_r, self.b_c), np.float32)
        if lib().orc_get_block(self.h, i, j, _fp(out)) != 0:
            raise IndexError("no node at (%d, %d)" % (i, j))
        return out

    def u(self, i, j):
        out = np.empty((self.ns, self.b_c), np.float32)
        if lib().orc_get_u(self.h, i, j, _fp(out)) != 0:
            raise IndexError("no node")
        return out

    def v(self, i, j):
        out = np.empty((self.nsc, self.b_r), np.float32)
        if lib().orc_get_v(self.h, i, j, _fp(out)) != 0:
            raise IndexError("no node")
        return out

    def set_block(self, i, j, data):
        data = _f32(data).reshape(self.b_r, self.b_c)
        if lib().orc_set_block(self.h, i, j, _fp(data)) != 0:
            raise IndexError("no node")

    def corrupt_block(self, i, j, seed, layer, iteration, density, amplitude):
        """Adds the sparse fault matrix to stored block (i, j); returns the number of elements changed."""
        q32 = min(int(density * 4294967296.0), 0xFFFFFFFF)
        n = int(lib().orc_corrupt_block(self.h, i, j, seed, layer, iteration, q32, C.c_float(amplitude)))
        if n < 0:
            raise IndexError("no node")
        return n

    def regenerate_block(self, i, j, along):
        rc = int(lib().orc_regenerate_block(self.h, i, j, along))
        if rc != 0:
            raise ValueError("block (%d, %d) cannot be regenerated along %d (code %d)" % (i, j, along, rc))

    def checkpoint_save(self):
        """Copies the stored state (coded blocks, inner checksums) aside."""
        if lib().orc_checkpoint_save(self.h) != 0:
            raise MemoryError("checkpoint")

    def checkpoint_restore(self):
        """Puts the last checkpoint back (the paper's answer to an uncorrectable pattern)."""
        if lib().orc_checkpoint_restore(self.h) != 0:
            raise RuntimeError("no checkpoint has been taken")

    def encode_x(self, X):
        X = _f32(X).reshape(-1, self.n_in)
        out = np.empty((X.shape[0], self.Nn * self.b_c), np.float32)
        lib().orc_encode_x(self.h, _fp(X), X.shape[0], _fp(out))
        return out

    def encode_delta(self, D):
        D = _f32(D).reshape(-1, self.n_out)
        out = np.empty((D.shape[0], self.M * self.b_r), np.float32)
        lib().orc_encode_delta(self.h, _fp(D), D.shape[0], _fp(out))
        return out

    def forward_products(self, X):
        X = _f32(X).reshape(-1, self.n_in)
        B = X.shape[0]
        Y = np.empty((self.n, self.M, self.b_r, B), np.float32)
        lib().orc_forward_products(self.h, _fp(X), B, _fp(Y))
        return Y

    def backward_products(self, D):
        D = _f32(D).reshape(-1, self.n_out)
        B = D.shape[0]
        Z = np.empty((self.m, self.Nn, self.b_c, B), np.float32)
        lib().orc_backward_products(self.h, _fp(D), B, _fp(Z))
        return Z

    def inject(self, phase, fault, iteration, Y):
        """Corrupts Y in place; returns the per-codeword injected masks."""
        assert Y.dtype == np.float32 and Y.flags.c_contiguous
        inj = (C.c_uint64 * 64)()
        lib().orc_inject(self.h, phase, C.byref(fault), iteration, _fp(Y), Y.shape[-1], inj)
        return [int(x) for x in inj]

    def detect_decode(self, phase, Y, V, Yclean=None, injected=None):
        """Corrects Y in place; returns the report."""
        assert Y.dtype == np.float32 and Y.flags.c_contiguous
        B = Y.shape[-1]
        V = _f32(V).reshape(B, -1)
        rep = Report()
        inj = None
        if injected is not None:
            inj = (C.c_uint64 * 64)(*injected)
        yc = None
        if Yclean is not None:
            Yclean = _f32(Yclean)
            yc = _fp(Yclean)
        lib().orc_detect_decode(self.h, phase, _fp(Y), _fp(V), B, yc, inj, C.byref(rep))
        return rep

    def forward(self, X, fault=None, iteration=0):
        X = _f32(X).reshape(-1, self.n_in)
        B = X.shape[0]
        S = np.zeros((B, self.n_out), np.float32)
        rep = Report()
        lib().orc_forward(self.h, _fp(X), B, None if fault is None else C.byref(fault), iteration,
                          _fp(S), C.byref(rep))
        return S, rep

    def update(self, D, X, lr):
        D = _f32(D).reshape(-1, self.n_out)
        X = _f32(X).reshape(-1, self.n_in)
        lib().orc_update(self.h, _fp(D), _fp(X), D.shape[0], lr)

    def backward_update(self, D, X, lr, fault=None, iteration=0):
        D = _f32(D).reshape(-1, self.n_out)
        X = _f32(X).reshape(-1, self.n_in)
        B = D.shape[0]
        Cc = np.zeros((B, self.n_in), np.float32)
        rep = Report()
        lib().orc_backward_update(self.h, _fp(D), _fp(X), B, lr,
                                  None if fault is None else C.byref(fault), iteration, _fp(Cc),
                                  C.byref(rep))
        return Cc, rep

    def decode_weights(self):
        W = np.empty((self.n_out, self.n_in), np.float32)
        lib().orc_decode_weights(self.h, _fp(W))
        return W

    def set_small_faults(self, plan):
        """Soft errors in the small steps (encoding, input copies, detection, decoding) of every later call; None: off."""
        self._small = plan
        lib().orc_layer_set_small_faults(self.h, None if plan is None else C.byref(plan))

    def code_conditioning(self, phase):
        """(worst condition number, worst ||A^-1||, worst error amplification) over the erasure sub-systems."""
        out = (C.c_double * 3)()
        lib().orc_code_conditioning(self.h, phase, out)
        return float(out[0]), float(out[1]), float(out[2])

    def check_invariance(self):
        return float(lib().orc_check_invariance(self.h))


class Net:
    def __init__(self, layers, activation=ACT_IDENTITY, loss=LOSS_MSE_MEAN):
        self.layers = list(layers)
        arr = (C.c_void_p * len(layers))(*[l.h for l in layers])
        self.h = lib().orc_net_create(arr, len(layers), activation, loss)
        if not self.h:
            raise ValueError("layer shapes do not chain")
        self.loss_kind = loss

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_net_free(self.h)
            self.h = None

    def step(self, X, target, lr, faults=None, iteration=0):
        """Returns (loss, last-layer output, [2L reports])."""
        L = len(self.layers)
        X = _f32(X).reshape(-1, self.layers[0].n_in)
        B = X.shape[0]
        if self.loss_kind == LOSS_MSE_MEAN:
            tgt = _f32(target).reshape(B, -1)
        else:
            tgt = np.ascontiguousarray(target, dtype=np.int32).reshape(B)
        reps = (Report * (2 * L))()
        farr = None
        if faults is not None:
            farr = (Fault * L)(*faults)
        loss = C.c_float()
        out = np.empty((B, self.layers[-1].n_out), np.float32)
        lib().orc_step(self.h, _fp(X), tgt.ctypes.data_as(C.c_void_p), B, lr, farr, iteration, reps,
                       C.byref(loss), _fp(out))
        return float(loss.value), out, list(reps)
