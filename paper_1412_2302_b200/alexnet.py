"""Thin Python binding of the C ABI in include/alexnet.h (argument marshalling only).

PyTorch is used for device memory, pinned host memory and streams; every step
of the training path runs inside the CUDA library.  There is no CPU fallback:
if the library has not been built, importing a handle fails loudly.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from . import build as _build

OK, ERR_ARG, ERR_CUDA, ERR_STATE, ERR_DEVICE_TIMEOUT, ERR_NOMEM = 0, -1, -2, -3, -4, -5
FLAG_LRN_ALPHA_DIV_N, FLAG_WD_ON_BIASES, FLAG_INVERTED_DROPOUT, FLAG_FUSED_FC_UPDATE = 1, 2, 4, 8
FLAG_NO_CTA_PAIRS, FLAG_ALL_CTA_PAIRS, FLAG_SHARED_REPLICA_WEIGHTS, FLAG_FC_CHAIN = 16, 32, 64, 128

TENSORS = ["CROPFLIP", "X0", "A1", "N1", "P1", "ARG1", "A2", "N2", "P2", "ARG2", "A3", "A4", "A5", "P5", "ARG5",
           "F6", "F7", "Z", "M6", "M7", "DZ", "DF7", "DF6", "DP5", "DA5", "DA4", "DA3", "DP2", "DN2", "DA2",
           "DP1", "DN1", "DA1", "LOSS", "DX0"]
T = {n: i for i, n in enumerate(TENSORS)}
OPS = ["CONV1_FWD", "CONV2_FWD", "CONV3_FWD", "CONV4_FWD", "CONV5_FWD",
       "CONV2_BWD_DATA", "CONV3_BWD_DATA", "CONV4_BWD_DATA", "CONV5_BWD_DATA",
       "CONV1_BWD_WEIGHT", "CONV2_BWD_WEIGHT", "CONV3_BWD_WEIGHT", "CONV4_BWD_WEIGHT", "CONV5_BWD_WEIGHT",
       "FC6_FWD", "FC7_FWD", "FC8_FWD", "FC6_BWD_DATA", "FC7_BWD_DATA", "FC8_BWD_DATA",
       "FC6_BWD_WEIGHT", "FC7_BWD_WEIGHT", "FC8_BWD_WEIGHT",
       "LRN1_FWD", "LRN2_FWD", "LRN1_BWD", "LRN2_BWD", "POOL1_FWD", "POOL2_FWD", "POOL5_FWD",
       "POOL1_BWD", "POOL2_BWD", "POOL5_BWD", "SOFTMAX", "UPDATE", "AVERAGE", "PREPROCESS", "CONV1_BWD_DATA",
       "LRN1_POOL1_FWD", "LRN2_POOL2_FWD", "POOL1_LRN1_BWD", "POOL2_LRN2_BWD", "UPDATE_AVERAGE", "SCALE_REFRESH", "FC_CHAIN_FWD"]
OP = {n: i for i, n in enumerate(OPS)}

EXPORTS = ["alexnet_param_count", "alexnet_workspace_bytes", "alexnet_create", "alexnet_destroy",
           "alexnet_load_batch_async", "alexnet_train_step", "alexnet_loss_async", "alexnet_replica_average", "alexnet_get_params",
           "alexnet_set_params", "alexnet_eval_batch", "alexnet_tensor_size", "alexnet_get_tensor", "alexnet_set_tensor", "alexnet_run_op",
           "alexnet_launch_count", "alexnet_profile", "alexnet_profile_read", "alexnet_sync", "alexnet_last_error", "alexnet_bias_grad_noalloc", "alexnet_loader_ring_bytes",
           "alexnet_loader_create", "alexnet_loader_next", "alexnet_loader_release", "alexnet_loader_destroy",
           "alexnet_forward_backward", "alexnet_apply_update", "alexnet_update_and_average", "alexnet_param_regions",
           "alexnet_scale_and_refresh", "alexnet_create_error", "alexnet_debug_expire_wait", "alexnet_set_color_augmentation", "alexnet_average_received", "alexnet_param_layout",
           "alexnet_stream_wait_fc_gradients", "alexnet_timeline_read"]


class Config(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("replicas", ctypes.c_int32), ("seed", ctypes.c_uint64),
                ("lr", ctypes.c_float), ("momentum", ctypes.c_float), ("weight_decay", ctypes.c_float),
                ("lrn_size", ctypes.c_int32), ("lrn_alpha", ctypes.c_float), ("lrn_beta", ctypes.c_float),
                ("lrn_k", ctypes.c_float), ("dropout_p", ctypes.c_float), ("init_std", ctypes.c_float),
                ("flags", ctypes.c_uint32)]


class AlexNetError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"alexnet error {code}: {msg}")
        self.code = code


_lib = None


def load_library():
    """dlopen the in-tree CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB):
        raise RuntimeError(f"{_build.LIB} is missing: run `python -m paper_1412_2302_b200.build` "
                           "(there is no CPU fallback)")
    L = ctypes.CDLL(_build.LIB)
    vp, sz, i32, u64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint64
    L.alexnet_param_count.restype = sz
    L.alexnet_workspace_bytes.restype = sz
    L.alexnet_workspace_bytes.argtypes = [ctypes.POINTER(Config)]
    L.alexnet_create.argtypes = [ctypes.POINTER(Config), vp, sz, vp, vp, vp, ctypes.POINTER(vp)]
    L.alexnet_destroy.argtypes = [vp]
    L.alexnet_load_batch_async.argtypes = [vp, i32, vp, vp, u64]
    L.alexnet_train_step.argtypes = [vp, i32, vp]
    L.alexnet_loss_async.argtypes = [vp, i32, vp]
    L.alexnet_replica_average.argtypes = [vp]
    L.alexnet_forward_backward.argtypes = [vp, i32, vp]
    L.alexnet_apply_update.argtypes = [vp, i32, ctypes.c_float]
    L.alexnet_update_and_average.argtypes = [vp]
    L.alexnet_param_regions.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(sz)]
    L.alexnet_scale_and_refresh.argtypes = [vp, i32, ctypes.c_float]
    L.alexnet_create_error.restype = ctypes.c_char_p
    L.alexnet_create_error.argtypes = []
    L.alexnet_debug_expire_wait.argtypes = [vp, ctypes.c_longlong]
    L.alexnet_set_color_augmentation.argtypes = [vp, vp, vp, ctypes.c_float]
    L.alexnet_average_received.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), i32, i32]
    L.alexnet_param_layout.argtypes = [vp, ctypes.POINTER(sz), ctypes.POINTER(sz), ctypes.POINTER(sz)]
    L.alexnet_stream_wait_fc_gradients.argtypes = [vp, vp]
    L.alexnet_timeline_read.argtypes = [vp, i32]
    L.alexnet_eval_batch.argtypes = [vp, i32, vp, vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32),
                                     ctypes.POINTER(ctypes.c_float)]
    L.alexnet_get_params.argtypes = [vp, i32, i32, vp, sz]
    L.alexnet_set_params.argtypes = [vp, i32, i32, vp, sz]
    L.alexnet_tensor_size.restype = sz
    L.alexnet_tensor_size.argtypes = [vp, i32]
    L.alexnet_get_tensor.argtypes = [vp, i32, i32, vp, sz]
    L.alexnet_set_tensor.argtypes = [vp, i32, i32, vp, sz]
    L.alexnet_run_op.argtypes = [vp, i32, i32, i32]
    L.alexnet_launch_count.restype = u64
    L.alexnet_launch_count.argtypes = [vp]
    L.alexnet_profile.argtypes = [vp, i32]
    L.alexnet_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(u64)]
    L.alexnet_sync.argtypes = [vp]
    L.alexnet_last_error.restype = ctypes.c_char_p
    L.alexnet_last_error.argtypes = [vp]
    L.alexnet_loader_ring_bytes.restype = sz
    L.alexnet_loader_ring_bytes.argtypes = [ctypes.c_int32, ctypes.c_int32]
    L.alexnet_loader_create.argtypes = [vp, vp, u64, ctypes.c_int32, vp, sz, ctypes.c_int32, ctypes.c_int32, u64, ctypes.c_int32,
                                        ctypes.POINTER(vp)]
    L.alexnet_loader_next.argtypes = [vp, ctypes.c_int32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(u64)]
    L.alexnet_loader_release.argtypes = [vp]
    L.alexnet_loader_destroy.argtypes = [vp]
    L.alexnet_bias_grad_noalloc.argtypes = [vp, ctypes.c_int64, ctypes.c_int32, vp, vp, ctypes.c_char_p, sz]
    _lib = L
    return L


def _ptr(x):
    """Raw address of a torch tensor or numpy array."""
    if hasattr(x, "data_ptr"):
        return ctypes.c_void_p(x.data_ptr())
    return ctypes.c_void_p(x.ctypes.data)


class AlexNet:
    """One handle = `replicas` identically initialised AlexNets in one GPU's memory."""

    def __init__(self, batch, replicas=1, seed=14122302, lr=0.01, momentum=0.9, weight_decay=5e-4,
                 lrn_alpha=1e-4, lrn_beta=0.75, lrn_k=2.0, dropout_p=0.5, init_std=0.0, flags=0,
                 mean_image=None, device="cuda:0", compute_stream=None, copy_stream=None):
        import torch
        self._torch = torch
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.cfg = Config(batch, replicas, seed, lr, momentum, weight_decay, 5, lrn_alpha, lrn_beta, lrn_k,
                          dropout_p, init_std, flags)
        self.batch, self.replicas = batch, replicas
        nbytes = self.lib.alexnet_workspace_bytes(ctypes.byref(self.cfg))
        if nbytes == 0:
            raise AlexNetError(ERR_ARG, "invalid configuration")
        self.arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 1023) // 1024 * 1024
        self.compute_stream = compute_stream or torch.cuda.Stream(self.device)
        self.copy_stream = copy_stream or torch.cuda.Stream(self.device)
        mean = None if mean_image is None else np.ascontiguousarray(mean_image, np.float32)
        h = ctypes.c_void_p()
        rc = self.lib.alexnet_create(ctypes.byref(self.cfg), ctypes.c_void_p(base), nbytes,
                                     None if mean is None else _ptr(mean),
                                     ctypes.c_void_p(self.compute_stream.cuda_stream),
                                     ctypes.c_void_p(self.copy_stream.cuda_stream), ctypes.byref(h))
        if rc != OK:
            raise AlexNetError(rc, self.lib.alexnet_create_error().decode() or "alexnet_create failed")
        self.h = h
        self.param_count = int(self.lib.alexnet_param_count())
        self._keep = []

    def _ck(self, rc):
        if rc != OK:
            raise AlexNetError(rc, self.lib.alexnet_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            self.lib.alexnet_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the path
    def load_batch_async(self, replica, images, labels, step):
        """images uint8 [B,256,256,3], labels int32 [B]; pinned-host or device torch tensors (or numpy)."""
        self._keep = self._keep[-8:] + [(images, labels)]
        self._ck(self.lib.alexnet_load_batch_async(self.h, replica, _ptr(images), _ptr(labels), int(step)))

    def train_step(self, replica=0, want_loss=False):
        if want_loss:
            loss = ctypes.c_float()
            self._ck(self.lib.alexnet_train_step(self.h, replica, ctypes.byref(loss)))
            return loss.value
        self._ck(self.lib.alexnet_train_step(self.h, replica, None))
        return None

    def loss_async(self, replica, out):
        """Queue the copy of the last step's mean loss into `out` (one float32, pinned host or device tensor) on the
        compute stream; the value is there once that stream has reached this point."""
        self._keep = self._keep[-8:] + [out]
        self._ck(self.lib.alexnet_loss_async(self.h, replica, _ptr(out)))

    def eval_batch(self, replica, images, labels):
        """(top-1 count, top-5 count, mean loss) of one minibatch: forward pass on the centre crop, no dropout mask."""
        t1, t5, loss = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_float()
        self._keep = self._keep[-8:] + [(images, labels)]
        self._ck(self.lib.alexnet_eval_batch(self.h, replica, _ptr(images), _ptr(labels), ctypes.byref(t1), ctypes.byref(t5),
                                             ctypes.byref(loss)))
        return t1.value, t5.value, loss.value

    def replica_average(self):
        self._ck(self.lib.alexnet_replica_average(self.h))

    def forward_backward(self, replica=0, want_loss=False):
        """train_step without the update: the gradient stays pending (apply_update / update_and_average consume it)."""
        if want_loss:
            loss = ctypes.c_float()
            self._ck(self.lib.alexnet_forward_backward(self.h, replica, ctypes.byref(loss)))
            return loss.value
        self._ck(self.lib.alexnet_forward_backward(self.h, replica, None))
        return None

    def apply_update(self, replica=0, grad_scale=1.0):
        self._ck(self.lib.alexnet_apply_update(self.h, replica, float(grad_scale)))

    def update_and_average(self):
        self._ck(self.lib.alexnet_update_and_average(self.h))

    def scale_and_refresh(self, replica=0, scale=1.0):
        self._ck(self.lib.alexnet_scale_and_refresh(self.h, replica, float(scale)))

    def average_received(self, replica, recv_w, recv_v, self_rank):
        """Average the replica's parameters and momentum with the copies received from the other replicas: recv_w / recv_v
        are lists with one fp32 CUDA tensor per rank (entry self_rank may be None: the replica's own arrays stand there)."""
        n = len(recv_w)
        pw, pv = (ctypes.c_void_p * n)(), (ctypes.c_void_p * n)()
        for r in range(n):
            pw[r] = None if r == self_rank or recv_w[r] is None else recv_w[r].data_ptr()
            pv[r] = None if r == self_rank or recv_v[r] is None else recv_v[r].data_ptr()
        self._keep = self._keep[-8:] + [(recv_w, recv_v)]
        self._ck(self.lib.alexnet_average_received(self.h, replica, pw, pv, n, int(self_rank)))

    def fc_range(self):
        """(begin, end) of the FC weights inside the arrays of param_views, in floats."""
        b, e = ctypes.c_size_t(), ctypes.c_size_t()
        self._ck(self.lib.alexnet_param_layout(self.h, ctypes.byref(b), ctypes.byref(e), None))
        return int(b.value), int(e.value)

    def stream_wait_fc_gradients(self, stream):
        """Make `stream` (a torch.cuda.Stream) wait until the FC weight gradients of the backward pass issued last exist."""
        self._ck(self.lib.alexnet_stream_wait_fc_gradients(self.h, ctypes.c_void_p(stream.cuda_stream)))

    def param_views(self, replica=0):
        """(w, v, g): fp32 torch views of the replica's parameter, momentum and gradient arrays inside the arena (the
        library's internal order, zero padded), for collectives between processes; no copy is made."""
        w, v, g, n = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_size_t()
        self._ck(self.lib.alexnet_param_regions(self.h, replica, ctypes.byref(w), ctypes.byref(v), ctypes.byref(g), ctypes.byref(n)))
        base = self.arena.data_ptr()
        out = []
        for p in (w, v, g):
            off = p.value - base
            out.append(self.arena[off:off + 4 * n.value].view(self._torch.float32))
        return tuple(out)

    def set_color_augmentation(self, eigvec=None, eigval=None, sigma=0.0):
        """Intensity augmentation of training loads: eigvec (3,3), eigval (3,) of the data set's RGB values; sigma 0 = off."""
        if sigma == 0:
            self._ck(self.lib.alexnet_set_color_augmentation(self.h, None, None, 0.0))
            return
        ev = np.ascontiguousarray(eigvec, np.float32).reshape(3, 3)
        el = np.ascontiguousarray(eigval, np.float32).reshape(3)
        self._ck(self.lib.alexnet_set_color_augmentation(self.h, _ptr(ev), _ptr(el), float(sigma)))

    def debug_expire_wait(self, budget_cycles=2_000_000):
        self._ck(self.lib.alexnet_debug_expire_wait(self.h, int(budget_cycles)))

    def sync(self):
        self._ck(self.lib.alexnet_sync(self.h))

    # ---- parameters, tensors, single operations
    def get_params(self, replica=0, which=0):
        out = np.empty(self.param_count, np.float32)
        self._ck(self.lib.alexnet_get_params(self.h, replica, which, _ptr(out), out.size))
        return out

    def set_params(self, values, replica=0, which=0):
        v = np.ascontiguousarray(values, np.float32)
        self._ck(self.lib.alexnet_set_params(self.h, replica, which, _ptr(v), v.size))

    def tensor_size(self, name):
        return int(self.lib.alexnet_tensor_size(self.h, T[name]))

    def get_tensor(self, name, replica=0):
        out = np.empty(self.tensor_size(name), np.float32)
        self._ck(self.lib.alexnet_get_tensor(self.h, replica, T[name], _ptr(out), out.size))
        return out

    def set_tensor(self, name, values, replica=0):
        v = np.ascontiguousarray(values, np.float32).ravel()
        self._ck(self.lib.alexnet_set_tensor(self.h, replica, T[name], _ptr(v), v.size))

    def run_op(self, name, replica=0, iters=1):
        self._ck(self.lib.alexnet_run_op(self.h, replica, OP[name], iters))

    def profile(self, enable):
        self._ck(self.lib.alexnet_profile(self.h, 1 if enable else 0))

    def profile_read(self):
        """Per tensor-core kernel class (conv_kernel on convolutions, wgrad_kernel, gemm_kernel, conv_kernel on FC
        forward): summed device time in ms and launches since the last read, as two 4-tuples."""
        ms, n = (ctypes.c_double * 4)(), (ctypes.c_uint64 * 4)()
        self._ck(self.lib.alexnet_profile_read(self.h, ms, n))
        return tuple(ms), tuple(int(v) for v in n)

    @property
    def launch_count(self):
        return int(self.lib.alexnet_launch_count(self.h))


class Loader:
    """Worker thread that gathers minibatches from a dataset in host memory into a ring of staging slots
    (include/alexnet.h, alexnet_loader_*).  images: uint8 array [n,256,256,3]; labels: int32 [n] (numpy arrays or
    memory maps; they must outlive the loader).  The ring is allocated here: pinned through torch when pin=True."""

    def __init__(self, images, labels, batch, depth=3, seed=0, shuffle=True, pin=False, threads=2):
        self.lib = load_library()
        self.images, self.labels, self.batch = images, labels, batch
        nbytes = int(self.lib.alexnet_loader_ring_bytes(batch, depth))
        if nbytes == 0:
            raise AlexNetError(ERR_ARG, "invalid loader configuration")
        if pin:
            import torch
            self.ring = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
            ring_ptr = self.ring.data_ptr()
        else:
            self.ring = np.empty(nbytes, np.uint8)
            ring_ptr = self.ring.ctypes.data
        h = ctypes.c_void_p()
        rc = self.lib.alexnet_loader_create(_ptr(images), _ptr(labels), int(images.shape[0]), batch, ctypes.c_void_p(ring_ptr),
                                            nbytes, depth, threads, int(seed), 1 if shuffle else 0, ctypes.byref(h))
        if rc != OK:
            raise AlexNetError(rc, "alexnet_loader_create failed")
        self.h = h

    def next(self, timeout_ms=10000):
        """(images, labels, batch index): numpy views into the ring slot, valid until release()."""
        pi, pl, idx = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_uint64()
        rc = self.lib.alexnet_loader_next(self.h, int(timeout_ms), ctypes.byref(pi), ctypes.byref(pl), ctypes.byref(idx))
        if rc != OK:
            raise AlexNetError(rc, "loader: no batch (time-out, or every slot is held)")
        img = np.ctypeslib.as_array(ctypes.cast(pi, ctypes.POINTER(ctypes.c_uint8)), shape=(self.batch, 256, 256, 3))
        lab = np.ctypeslib.as_array(ctypes.cast(pl, ctypes.POINTER(ctypes.c_int32)), shape=(self.batch,))
        return img, lab, int(idx.value)

    def release(self):
        rc = self.lib.alexnet_loader_release(self.h)
        if rc != OK:
            raise AlexNetError(rc, "loader: nothing to release")

    def close(self):
        if getattr(self, "h", None):
            self.lib.alexnet_loader_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bias_grad_noalloc(dy, db, stream=None):
    """db[c] = sum_rows dy[row][c] through the entry point that allocates nothing.

    dy: CUDA bf16 tensor [rows, channels] (contiguous); db: CUDA fp32 tensor
    [channels], written in place.  For callers that must not allocate device
    memory (see include/alexnet.h); channels is limited to 4096.  Raises
    AlexNetError with the library's message when the sizes are rejected."""
    lib = load_library()
    msg = ctypes.create_string_buffer(256)
    rows, ch = int(dy.shape[0]), int(dy.shape[1])
    rc = lib.alexnet_bias_grad_noalloc(_ptr(dy), rows, ch, _ptr(db),
                                       ctypes.c_void_p(stream.cuda_stream if stream is not None else 0), msg, 256)
    if rc != OK:
        raise AlexNetError(rc, msg.value.decode())
