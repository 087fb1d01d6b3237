"""Thin Python binding of libcodenet.so: argument marshalling only.

Every function here has the name of the C entry point it calls (``include/codenet.h``); torch
is used for device memory and the current stream, nothing is computed in Python.  Loading
fails loudly if the CUDA library has not been built -- there is no CPU path.
"""
import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

F32, BF16 = 0, 1
MATH_FFMA, MATH_TF32, MATH_BF16 = 0, 1, 2
LOCATE_NONE, LOCATE_SYNDROME, LOCATE_NODECHECK, LOCATE_OFF, LOCATE_JOINT = 0, 1, 2, 3, 4
FAULT_NONE, FAULT_BERNOULLI, FAULT_EXACTLY_ONE = 0, 1, 2
PHASE_FWD, PHASE_BWD = 0, 1
CLEAN, CORRECTED, FALLBACK, FAILED, TIMEOUT, DISAGREE = 0, 1, 2, 3, 4, 5
PHASE_ENCODE, PHASE_INPUT, PHASE_CHECK, PHASE_DECODE = 2, 3, 4, 5
ACT_IDENTITY, ACT_RELU = 0, 1
LOSS_MSE_MEAN, LOSS_SOFTMAX_CE = 0, 1
MAX_NODES = 64


class LayerDesc(C.Structure):
    _fields_ = [("n_out", C.c_int32), ("n_in", C.c_int32), ("m", C.c_int32), ("n", C.c_int32),
                ("r_row", C.c_int32), ("r_col", C.c_int32), ("dtype", C.c_int32), ("math", C.c_int32),
                ("batch_max", C.c_int32), ("locate_mode", C.c_int32), ("check_rows", C.c_int32),
                ("check_cols", C.c_int32),
                ("P_row", C.POINTER(C.c_float)), ("P_col", C.POINTER(C.c_float)),
                ("tau_rel", C.c_float), ("tau_abs", C.c_float)]


class Fault(C.Structure):
    _fields_ = [("seed", C.c_uint32), ("layer", C.c_uint32), ("mode", C.c_uint32),
                ("p_q32", C.c_uint32), ("sigma", C.c_float), ("iteration_dev", C.c_void_p)]


class SmallFaults(C.Structure):
    _fields_ = [("seed", C.c_uint32), ("layer", C.c_uint32), ("p_encode_q32", C.c_uint32), ("p_input_q32", C.c_uint32),
                ("p_check_q32", C.c_uint32), ("p_decode_q32", C.c_uint32), ("sigma", C.c_float),
                ("iteration_dev", C.c_void_p)]


class Report(C.Structure):
    _fields_ = [("status", C.c_uint32), ("n_detected_cw", C.c_uint32),
                ("n_flagged_nodes", C.c_uint32), ("n_fallback_cw", C.c_uint32),
                ("detected_mask", C.c_uint64), ("flagged_mask", C.c_uint64 * MAX_NODES),
                ("injected_mask", C.c_uint64 * MAX_NODES),
                ("min_margin_hit", C.c_float), ("max_margin_clean", C.c_float)]

    def decisions(self):
        return (int(self.status), int(self.n_detected_cw), int(self.n_flagged_nodes),
                int(self.n_fallback_cw), int(self.detected_mask),
                tuple(int(x) for x in self.flagged_mask), tuple(int(x) for x in self.injected_mask))


REPORT_BYTES = C.sizeof(Report)

_lib = None


class CodenetError(RuntimeError):
    pass


def lib():
    """Load libcodenet.so (building it first if the sources are newer)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    if not os.path.exists(path):
        raise CodenetError("libcodenet.so is missing: run paper_1903_01042_b200/build.py")
    L = C.CDLL(path)
    vp, ip, fl = C.c_void_p, C.c_int, C.c_float
    L.codenet_strerror.restype = C.c_char_p
    L.codenet_strerror.argtypes = [ip]
    L.codenet_launch_count.restype = C.c_uint64
    L.codenet_profile_enable.argtypes = [ip]
    L.codenet_profile_enable.restype = ip
    L.codenet_profile_read.argtypes = [ip, C.POINTER(C.c_float), C.POINTER(C.c_uint64)]
    L.codenet_profile_read.restype = ip
    L.codenet_encode_layer.argtypes = [C.POINTER(LayerDesc), vp, vp, C.POINTER(vp)]
    L.codenet_forward.argtypes = [vp, vp, ip, C.POINTER(Fault), vp, vp, vp]
    L.codenet_backward_update.argtypes = [vp, vp, vp, ip, fl, C.POINTER(Fault), vp, vp, vp]
    L.codenet_backward_update_next.argtypes = [vp, vp, vp, ip, fl, C.POINTER(Fault), vp, vp, vp, vp]
    L.codenet_backward_update_forward_next.argtypes = [vp, vp, vp, ip, fl, C.POINTER(Fault), vp, vp, vp,
                                                       C.POINTER(Fault), vp, vp, vp]
    L.codenet_net_set_next_input.argtypes = [vp, vp]
    L.codenet_net_set_lookahead.argtypes = [vp, ip]
    L.codenet_net_set_lookahead.restype = ip
    L.codenet_net_set_iteration_counter.argtypes = [vp, vp]
    L.codenet_net_set_iteration_counter.restype = ip
    L.codenet_net_capture_step.argtypes = [vp, vp, vp, ip, fl, C.POINTER(Fault), vp, vp, vp, vp, C.POINTER(ip)]
    L.codenet_net_capture_steps.argtypes = [vp, ip, C.POINTER(vp), C.POINTER(vp), ip, fl, C.POINTER(Fault), vp, ip,
                                            vp, ip, vp, vp, C.POINTER(ip)]
    L.codenet_net_replay.argtypes = [vp, ip, vp]
    L.codenet_detect_decode.argtypes = [vp, ip, vp, vp, ip, vp, vp]
    L.codenet_net_create.argtypes = [C.POINTER(vp), ip, ip, ip, C.POINTER(vp)]
    L.codenet_step.argtypes = [vp, vp, vp, ip, fl, C.POINTER(Fault), vp, vp, vp]
    L.codenet_net_output.argtypes = [vp, vp, ip, vp]
    L.codenet_decode_weights.argtypes = [vp, vp, vp]
    L.codenet_check_invariance.argtypes = [vp, vp, vp]
    L.codenet_matvec_noalloc.argtypes = [vp, ip, ip, ip, vp, vp, vp]
    L.codenet_matvec_noalloc.restype = ip
    L.codenet_corrupt_block.argtypes = [vp, ip, ip, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, fl, vp]
    L.codenet_regenerate_block.argtypes = [vp, ip, ip, ip, vp]
    L.codenet_checkpoint_save.argtypes = [vp, vp]
    L.codenet_checkpoint_restore.argtypes = [vp, vp]
    L.codenet_get_block.argtypes = [vp, ip, ip, vp, vp]
    L.codenet_get_checksums.argtypes = [vp, ip, ip, vp, vp, vp]
    L.codenet_layer_dims.argtypes = [vp, C.POINTER(C.c_int32)]
    L.codenet_code_conditioning.argtypes = [vp, ip, C.POINTER(C.c_double)]
    L.codenet_code_conditioning.restype = ip
    L.codenet_layer_set_small_faults.argtypes = [vp, C.POINTER(SmallFaults)]
    L.codenet_layer_set_small_faults.restype = ip
    L.codenet_set_wait_limit.argtypes = [C.c_uint64, vp]
    L.codenet_set_wait_limit.restype = ip
    L.codenet_withhold_tile_loads.argtypes = [ip, vp]
    L.codenet_withhold_tile_loads.restype = ip
    L.codenet_reset_timeout.argtypes = [vp, vp]
    L.codenet_reset_timeout.restype = ip
    L.codenet_free_layer.argtypes = [vp]
    L.codenet_free_layer.restype = None
    L.codenet_free_net.argtypes = [vp]
    L.codenet_free_net.restype = None
    for name in ("codenet_encode_layer", "codenet_forward", "codenet_backward_update",
                 "codenet_detect_decode", "codenet_net_create", "codenet_step",
                 "codenet_decode_weights", "codenet_check_invariance", "codenet_get_block",
                 "codenet_layer_dims", "codenet_net_output", "codenet_get_checksums",
                 "codenet_backward_update_next", "codenet_backward_update_forward_next", "codenet_net_set_next_input", "codenet_net_capture_step",
                 "codenet_net_capture_steps",
                 "codenet_net_replay", "codenet_corrupt_block", "codenet_regenerate_block",
                 "codenet_checkpoint_save", "codenet_checkpoint_restore"):
        getattr(L, name).restype = ip
    _lib = L
    return L


def _check(rc):
    if rc != 0:
        raise CodenetError("libcodenet: %s (%d)" % (lib().codenet_strerror(rc).decode(), rc))


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def _dev_f32(t, shape=None):
    assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
    if shape is not None:
        assert tuple(t.shape) == tuple(shape), (tuple(t.shape), tuple(shape))
    return t


KERNEL_FORWARD, KERNEL_BACKWARD_UPDATE, KERNEL_BACKWARD, KERNEL_UPDATE, KERNEL_REGENERATE = 0, 1, 2, 3, 4


def profile_enable(on):
    """codenet_profile_enable."""
    _check(lib().codenet_profile_enable(1 if on else 0))


def profile_read(kernel):
    """codenet_profile_read: (total milliseconds, launches) of one streaming kernel."""
    ms = C.c_float()
    n = C.c_uint64()
    _check(lib().codenet_profile_read(kernel, C.byref(ms), C.byref(n)))
    return float(ms.value), int(n.value)


def launch_count():
    return int(lib().codenet_launch_count())


def strerror(code):
    return lib().codenet_strerror(code).decode()


def make_fault(seed=0, layer=0, mode=FAULT_NONE, p=0.0, sigma=10.0, iteration_dev=None):
    """Injection plan; ``iteration_dev`` is a 1-element uint32/int32 CUDA tensor (kept alive by the caller)."""
    p_q32 = min(int(p * 4294967296.0), 0xFFFFFFFF)
    return Fault(seed, layer, mode, p_q32, sigma, None if iteration_dev is None else iteration_dev.data_ptr())


def new_reports(count=1):
    """Device buffer for ``count`` reports."""
    return torch.zeros(count * REPORT_BYTES, dtype=torch.uint8, device="cuda")


def read_reports(buf):
    """Copy reports to the host (synchronises)."""
    host = buf.cpu().numpy().tobytes()
    n = len(host) // REPORT_BYTES
    return [Report.from_buffer_copy(host[k * REPORT_BYTES:(k + 1) * REPORT_BYTES]) for k in range(n)]


class Layer:
    """Handle of one coded layer (owns the device-side coded weights)."""

    def __init__(self, handle, desc, keep):
        self.h = handle
        self.desc = desc
        self._keep = keep
        dims = (C.c_int32 * 10)()
        _check(lib().codenet_layer_dims(self.h, dims))
        (self.b_r, self.b_c, self.M, self.Nn, self.T, self.ns, self.n_out_p, self.n_in_p, self.Tc,
         self.nsc) = [int(x) for x in dims]
        self.n_out, self.n_in, self.m, self.n = desc.n_out, desc.n_in, desc.m, desc.n
        self.r_row, self.r_col = desc.r_row, desc.r_col
        self.dtype = desc.dtype
        self.batch_max = desc.batch_max

    def free(self):
        if self.h:
            lib().codenet_free_layer(self.h)
            self.h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    def has_node(self, i, j):
        return i < self.M and j < self.Nn and (i < self.m or j < self.n)


def encode_layer(W_dev, m, n, r_row, r_col, P_row=None, P_col=None, dtype=None, math=MATH_FFMA,
                 batch_max=1, locate_mode=LOCATE_NODECHECK, check_rows=0, check_cols=0, tau_rel=None, tau_abs=1e-20):
    """codenet_encode_layer: W_dev is an (n_out, n_in) CUDA tensor, float32 or bfloat16."""
    assert W_dev.is_cuda and W_dev.is_contiguous() and W_dev.dim() == 2
    if dtype is None:
        dtype = BF16 if W_dev.dtype == torch.bfloat16 else F32
    assert (dtype == BF16) == (W_dev.dtype == torch.bfloat16)
    if tau_rel is None:
        tau_rel = 3e-2 if dtype == BF16 or math != MATH_FFMA else 1e-3
    pr = None if P_row is None else np.ascontiguousarray(P_row, dtype=np.float32).reshape(m, r_row)
    pc = None if P_col is None else np.ascontiguousarray(P_col, dtype=np.float32).reshape(n, r_col)
    fp = C.POINTER(C.c_float)
    d = LayerDesc(W_dev.shape[0], W_dev.shape[1], m, n, r_row, r_col, dtype, math, batch_max, locate_mode,
                  check_rows, check_cols, None if pr is None else pr.ctypes.data_as(fp),
                  None if pc is None else pc.ctypes.data_as(fp), tau_rel, tau_abs)
    h = C.c_void_p()
    _check(lib().codenet_encode_layer(C.byref(d), _ptr(W_dev), _stream(), C.byref(h)))
    return Layer(h, d, (pr, pc))


def forward(layer, X_dev, fault=None, S_dev=None, rep_dev=None):
    """codenet_forward: returns S_dev (B, n_out)."""
    B = X_dev.shape[0]
    _dev_f32(X_dev, (B, layer.n_in))
    if S_dev is None:
        S_dev = torch.empty((B, layer.n_out), dtype=torch.float32, device=X_dev.device)
    _dev_f32(S_dev, (B, layer.n_out))
    _check(lib().codenet_forward(layer.h, _ptr(X_dev), B, None if fault is None else C.byref(fault),
                                 _ptr(S_dev), _ptr(rep_dev), _stream()))
    return S_dev


def backward_update(layer, Delta_dev, X_dev, lr, fault=None, C_dev=None, rep_dev=None, X_next_dev=None):
    """codenet_backward_update / codenet_backward_update_next: returns C_dev (B, n_in); updates the
    coded weights; with X_next_dev also takes the next iteration's feedforward products."""
    B = X_dev.shape[0]
    _dev_f32(X_dev, (B, layer.n_in))
    _dev_f32(Delta_dev, (B, layer.n_out))
    if C_dev is None:
        C_dev = torch.empty((B, layer.n_in), dtype=torch.float32, device=X_dev.device)
    _dev_f32(C_dev, (B, layer.n_in))
    if X_next_dev is None:
        _check(lib().codenet_backward_update(layer.h, _ptr(Delta_dev), _ptr(X_dev), B, float(lr),
                                             None if fault is None else C.byref(fault), _ptr(C_dev),
                                             _ptr(rep_dev), _stream()))
    else:
        _dev_f32(X_next_dev, (B, layer.n_in))
        _check(lib().codenet_backward_update_next(layer.h, _ptr(Delta_dev), _ptr(X_dev), B, float(lr),
                                                  None if fault is None else C.byref(fault), _ptr(C_dev),
                                                  _ptr(rep_dev), _ptr(X_next_dev), _stream()))
    return C_dev


def backward_update_forward_next(layer, Delta_dev, X_dev, lr, X_next_dev, fault=None, fault_next=None, C_dev=None,
                                 rep_dev=None, S_next_dev=None, rep_next_dev=None):
    """codenet_backward_update_forward_next: this iteration's backward product, checks and update and the next
    iteration's whole forward stage; returns (C_dev, S_next_dev)."""
    B = X_dev.shape[0]
    _dev_f32(X_dev, (B, layer.n_in))
    _dev_f32(X_next_dev, (B, layer.n_in))
    _dev_f32(Delta_dev, (B, layer.n_out))
    if C_dev is None:
        C_dev = torch.empty((B, layer.n_in), dtype=torch.float32, device=X_dev.device)
    if S_next_dev is None:
        S_next_dev = torch.empty((B, layer.n_out), dtype=torch.float32, device=X_dev.device)
    _dev_f32(C_dev, (B, layer.n_in))
    _dev_f32(S_next_dev, (B, layer.n_out))
    _check(lib().codenet_backward_update_forward_next(
        layer.h, _ptr(Delta_dev), _ptr(X_dev), B, float(lr), None if fault is None else C.byref(fault), _ptr(C_dev),
        _ptr(rep_dev), _ptr(X_next_dev), None if fault_next is None else C.byref(fault_next), _ptr(S_next_dev),
        _ptr(rep_next_dev), _stream()))
    return C_dev, S_next_dev


def detect_decode(layer, phase, Y_dev, V_dev, rep_dev=None):
    """codenet_detect_decode: Y_dev [codeword][node][len][B] is corrected in place."""
    _dev_f32(Y_dev)
    _dev_f32(V_dev)
    B = Y_dev.shape[-1]
    _check(lib().codenet_detect_decode(layer.h, phase, _ptr(Y_dev), _ptr(V_dev), B, _ptr(rep_dev), _stream()))
    return Y_dev


class Net:
    def __init__(self, handle, layers, loss):
        self.h = handle
        self.layers = layers
        self.loss = loss

    def free(self):
        if self.h:
            lib().codenet_free_net(self.h)
            self.h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    def output(self, B):
        """codenet_net_output: the last layer's pre-loss output of the latest step."""
        out = torch.empty((B, self.layers[-1].n_out), dtype=torch.float32, device="cuda")
        _check(lib().codenet_net_output(self.h, _ptr(out), B, _stream()))
        return out


def net_create(layers, activation=ACT_IDENTITY, loss=LOSS_MSE_MEAN):
    """codenet_net_create."""
    arr = (C.c_void_p * len(layers))(*[l.h for l in layers])
    h = C.c_void_p()
    _check(lib().codenet_net_create(arr, len(layers), activation, loss, C.byref(h)))
    return Net(h, list(layers), loss)


def net_set_next_input(net, X_next_dev):
    """codenet_net_set_next_input: announce the next step's input (kept alive by the caller)."""
    _check(lib().codenet_net_set_next_input(net.h, _ptr(X_next_dev)))


def net_set_lookahead(net, on):
    """codenet_net_set_lookahead: use (default) or ignore announced next inputs."""
    _check(lib().codenet_net_set_lookahead(net.h, 1 if on else 0))


def net_set_iteration_counter(net, counter_dev):
    """codenet_net_set_iteration_counter: every step ends by advancing this device word (None: off)."""
    _check(lib().codenet_net_set_iteration_counter(net.h, _ptr(counter_dev)))


def net_capture_step(net, X_dev, target_dev, lr, faults=None, reps_dev=None, loss_dev=None, X_next_dev=None):
    """codenet_net_capture_step: record one step into a CUDA graph; returns its id."""
    B = X_dev.shape[0]
    _dev_f32(X_dev, (B, net.layers[0].n_in))
    farr = None
    if faults is not None:
        farr = (Fault * len(net.layers))(*faults)
    gid = C.c_int(-1)
    _check(lib().codenet_net_capture_step(net.h, _ptr(X_dev), _ptr(target_dev), B, float(lr), farr, _ptr(reps_dev),
                                          _ptr(loss_dev), _ptr(X_next_dev), _stream(), C.byref(gid)))
    return int(gid.value)


def net_capture_steps(net, X_devs, target_devs, lr, faults=None, reps_dev=None, reps_stride=0, loss_dev=None,
                      loss_stride=0, X_next_dev=None):
    """codenet_net_capture_steps: record len(X_devs) consecutive steps into one CUDA graph; returns its id."""
    B = X_devs[0].shape[0] if len(X_devs) else 0
    for x in X_devs:
        _dev_f32(x, (B, net.layers[0].n_in))
    n = len(X_devs)
    xs = (C.c_void_p * max(n, 1))(*[_ptr(x) for x in X_devs])
    ts = (C.c_void_p * max(n, 1))(*[_ptr(t) for t in target_devs])
    farr = None
    if faults is not None:
        farr = (Fault * len(net.layers))(*faults)
    gid = C.c_int(-1)
    _check(lib().codenet_net_capture_steps(net.h, n, xs, ts, B, float(lr), farr, _ptr(reps_dev), int(reps_stride),
                                           _ptr(loss_dev), int(loss_stride), _ptr(X_next_dev), _stream(),
                                           C.byref(gid)))
    return int(gid.value)


def net_replay(net, graph_id):
    """codenet_net_replay: enqueue one recorded step on the current stream."""
    _check(lib().codenet_net_replay(net.h, graph_id, _stream()))


def step(net, X_dev, target_dev, lr, faults=None, reps_dev=None, loss_dev=None):
    """codenet_step: one training iteration of the whole network."""
    B = X_dev.shape[0]
    _dev_f32(X_dev, (B, net.layers[0].n_in))
    assert target_dev.is_cuda and target_dev.is_contiguous()
    if net.loss == LOSS_SOFTMAX_CE:
        assert target_dev.dtype == torch.int32
    else:
        assert target_dev.dtype == torch.float32
    farr = None
    if faults is not None:
        farr = (Fault * len(net.layers))(*faults)
    _check(lib().codenet_step(net.h, _ptr(X_dev), _ptr(target_dev), B, float(lr), farr, _ptr(reps_dev),
                              _ptr(loss_dev), _stream()))


def decode_weights(layer, out=None):
    """codenet_decode_weights: the m x n data blocks as an (n_out, n_in) tensor."""
    dt = torch.bfloat16 if layer.dtype == BF16 else torch.float32
    if out is None:
        out = torch.empty((layer.n_out, layer.n_in), dtype=dt, device="cuda")
    _check(lib().codenet_decode_weights(layer.h, _ptr(out), _stream()))
    return out


def code_conditioning(layer, phase):
    """codenet_code_conditioning: (worst condition number, worst ||A^-1||, worst error amplification)."""
    out = (C.c_double * 3)()
    _check(lib().codenet_code_conditioning(layer.h, int(phase), out))
    return float(out[0]), float(out[1]), float(out[2])


def set_wait_limit(nanoseconds):
    _check(lib().codenet_set_wait_limit(int(nanoseconds), _stream()))


def withhold_tile_loads(on):
    _check(lib().codenet_withhold_tile_loads(1 if on else 0, _stream()))


def reset_timeout(layer):
    _check(lib().codenet_reset_timeout(layer.h, _stream()))


def make_small_faults(seed=0, layer=0, p_encode=0.0, p_input=0.0, p_check=0.0, p_decode=0.0, sigma=10.0,
                      iteration_dev=None):
    """Plan for soft errors in the small steps; ``iteration_dev`` as in make_fault."""
    q = lambda p: min(int(p * 4294967296.0), 0xFFFFFFFF)
    return SmallFaults(seed, layer, q(p_encode), q(p_input), q(p_check), q(p_decode), sigma,
                       None if iteration_dev is None else iteration_dev.data_ptr())


def set_small_faults(layer, plan):
    """codenet_layer_set_small_faults: applies to every later call on the layer; None switches it off."""
    layer._small = plan
    _check(lib().codenet_layer_set_small_faults(layer.h, None if plan is None else C.byref(plan)))


def check_invariance(layer):
    """codenet_check_invariance: returns the deviation as a Python float (synchronises)."""
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    _check(lib().codenet_check_invariance(layer.h, _ptr(out), _stream()))
    return float(out.item())


def corrupt_block(layer, i, j, seed, fault_layer, iteration, density, amplitude):
    """Adds the sparse fault matrix of the paper's experiment to stored block (i, j)."""
    q32 = min(int(density * 4294967296.0), 0xFFFFFFFF)
    _check(lib().codenet_corrupt_block(layer.h, int(i), int(j), C.c_uint32(seed), C.c_uint32(fault_layer),
                                       C.c_uint32(iteration), C.c_uint32(q32), C.c_float(amplitude), _stream()))


def regenerate_block(layer, i, j, along):
    """Rebuilds stored block (i, j) from the code of its block-column (along = 0) or block-row (along = 1)."""
    _check(lib().codenet_regenerate_block(layer.h, int(i), int(j), int(along), _stream()))


def checkpoint_save(layer):
    """codenet_checkpoint_save: copies the layer's coded blocks and inner checksums aside (device memory)."""
    _check(lib().codenet_checkpoint_save(layer.h, _stream()))


def checkpoint_restore(layer):
    """codenet_checkpoint_restore: puts the last checkpoint back (roll-back after an uncorrectable pattern)."""
    _check(lib().codenet_checkpoint_restore(layer.h, _stream()))


def get_block(layer, i, j):
    """codenet_get_block: stored coded block (i, j) as a (b_r, b_c) float tensor."""
    out = torch.empty((layer.b_r, layer.b_c), dtype=torch.float32, device="cuda")
    _check(lib().codenet_get_block(layer.h, i, j, _ptr(out), _stream()))
    return out


def get_checksums(layer, i, j):
    """codenet_get_checksums: (u, v) inner checksums of block (i, j)."""
    u = torch.empty((layer.ns, layer.b_c), dtype=torch.float32, device="cuda")
    v = torch.empty((layer.nsc, layer.b_r), dtype=torch.float32, device="cuda")
    _check(lib().codenet_get_checksums(layer.h, i, j, _ptr(u), _ptr(v), _stream()))
    return u, v


def matvec_noalloc(W_dev, n_blocks, x_dev, s_dev):
    """codenet_matvec_noalloc: s = W x with the library's fixed scratch, no allocation anywhere.

    The output tensor is the caller's too, so that this wrapper does not allocate either."""
    assert W_dev.is_cuda and W_dev.dtype == torch.float32 and W_dev.is_contiguous() and W_dev.dim() == 2
    rows, cols = W_dev.shape
    _dev_f32(x_dev)
    _dev_f32(s_dev)
    assert x_dev.numel() == cols and s_dev.numel() == rows
    _check(lib().codenet_matvec_noalloc(_ptr(W_dev), rows, cols, n_blocks, _ptr(x_dev), _ptr(s_dev), _stream()))
    return s_dev
