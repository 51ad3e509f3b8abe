"""ctypes binding of libsegtrain.so: the functions of include/seg.h under the same names,
plus `Segment`, a thin holder that marshals torch tensors into those calls.

Argument marshalling only: every step of the training path runs in the library's CUDA
kernels.  Importing this module without the built library raises; there is no CPU path.
"""
import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int32, c_uint64, c_void_p

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsegtrain.so")

SEG_OK = 0
SEG_FP32, SEG_TF32, SEG_BF16 = 0, 1, 2
SEG_SGD, SEG_SGD_MOMENTUM, SEG_ADAM = 0, 1, 2
SEG_LABEL_UNIFORM_KAPPA, SEG_LABEL_NORMAL = 0, 1
SEG_GEMM_AUTO, SEG_GEMM_SIMT, SEG_GEMM_TCGEN05 = 0, 1, 2
PRECISIONS = {"fp32": SEG_FP32, "tf32": SEG_TF32, "bf16": SEG_BF16}
OPTIMIZERS = {"sgd": SEG_SGD, "momentum": SEG_SGD_MOMENTUM, "adam": SEG_ADAM}
LABEL_DISTS = {"uniform_kappa": SEG_LABEL_UNIFORM_KAPPA, "normal": SEG_LABEL_NORMAL}
BACKENDS = {"auto": SEG_GEMM_AUTO, "simt": SEG_GEMM_SIMT, "tcgen05": SEG_GEMM_TCGEN05}
# kind numbers of seg_profile_get
KERNEL_KINDS = {0: "fwd_gemm", 1: "dgrad_gemm", 2: "wgrad_gemm", 3: "loss", 4: "wgrad_update_gemm", 5: "update", 6: "copy",
                7: "fwd_loss_dgrad"}
# order of the counters seg_product_launches returns (the last one counts a subset of tc_single + tc_pair)
PRODUCT_FAMILIES = ("tc_single", "tc_splitk", "tc_pair", "ffma", "fused_update")


class seg_config(Structure):
    _fields_ = [("n_layers", c_int32), ("widths", POINTER(c_int32)), ("n_classes", c_int32),
                ("is_final", c_int32), ("last_relu", c_int32), ("segment_id", c_int32),
                ("precision", c_int32), ("optimizer", c_int32),
                ("lr", c_float), ("momentum", c_float), ("beta1", c_float), ("beta2", c_float),
                ("eps", c_float), ("max_batch", c_int32), ("gemm_backend", c_int32),
                ("init_seed", c_uint64), ("stream", c_void_p)]


EXPORTS = {
    "seg_create": (c_int32, [POINTER(seg_config), POINTER(c_void_p)]),
    "seg_gen_labels": (c_int32, [c_void_p, c_uint64, c_int32, c_float]),
    "seg_train_step": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p]),
    "seg_train_step_label_input": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_void_p]),
    "seg_train_step_host": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_float)]),
    "seg_train_step_host_async": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_void_p]),
    "seg_forward": (c_int32, [c_void_p, c_void_p, c_int32, c_void_p]),
    "seg_recovery_step": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_void_p]),
    "seg_train_epochs": (c_int32, [c_void_p, c_void_p, c_void_p, ctypes.c_int64, c_int32, c_int32, c_void_p]),
    "seg_forward_dataset": (c_int32, [c_void_p, c_void_p, ctypes.c_int64, c_int32, c_void_p]),
    "seg_destroy": (c_int32, [c_void_p]),
    "seg_get_labels": (c_int32, [c_void_p, c_void_p]),
    "seg_set_labels": (c_int32, [c_void_p, c_void_p]),
    "seg_get_params": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p]),
    "seg_set_params": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p]),
    "seg_get_grads": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p]),
    "seg_get_opt_state": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p]),
    "seg_set_opt_state": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p]),
    "seg_get_step": (c_int32, [c_void_p, POINTER(c_uint64)]),
    "seg_set_step": (c_int32, [c_void_p, c_uint64]),
    "seg_get_activation": (c_int32, [c_void_p, c_int32, c_void_p]),
    "seg_mem_bytes": (c_int32, [c_void_p, POINTER(c_uint64), POINTER(c_uint64)]),
    "seg_launch_count": (c_int32, [c_void_p, POINTER(c_uint64)]),
    "seg_product_launches": (c_int32, [c_void_p, POINTER(c_uint64)]),
    "seg_poll_status": (c_int32, [c_void_p]),
    "seg_selftest_bounded_wait": (c_int32, [c_void_p, c_uint64]),
    "seg_handoff_copy": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_uint64]),
    "seg_device": (c_int32, [c_void_p, POINTER(c_int32)]),
    "seg_timer_start": (c_int32, [c_void_p]),
    "seg_timer_stop": (c_int32, [c_void_p]),
    "seg_timer_elapsed_ms": (c_int32, [c_void_p, POINTER(c_float)]),
    "seg_profile_enable": (c_int32, [c_void_p, c_int32]),
    "seg_profile_get": (c_int32, [c_void_p, c_int32, POINTER(c_uint64), POINTER(c_float)]),
    "seg_label_loss_noalloc": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32,
                                         c_void_p, c_void_p, c_void_p]),
    "seg_status_string": (c_char_p, [c_int32]),
    "seg_last_error": (c_char_p, [c_void_p]),
    "seg_build_info": (c_char_p, []),
}

_lib = None


def load():
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2403_11204_b200.build` "
                               "(there is no fallback path)")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


class SegError(RuntimeError):
    def __init__(self, status, detail=""):
        self.status = status
        msg = load().seg_status_string(status).decode()
        super().__init__(f"seg status {status}: {msg}" + (f" ({detail})" if detail else ""))


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def label_loss_noalloc(out, cls, sil, relu_mask, dz, loss_out, stream=None):
    """seg_label_loss_noalloc on torch CUDA tensors: the intermediate-label loss and its dZ for
    callers that must not allocate device memory (the library's static scratch is used).
    out [batch, n_p] fp32, cls [batch] int32, sil [n_classes, n_p] fp32; dz and loss_out are
    written.  Calls that may overlap on the GPU share the scratch and must be ordered."""
    import torch
    lib = load()
    for t in (out, cls, sil, dz):
        assert t.is_cuda and t.is_contiguous()
    assert out.dtype == torch.float32 and sil.dtype == torch.float32 and dz.dtype == torch.float32
    assert cls.dtype == torch.int32 and dz.shape == out.shape and sil.shape[1] == out.shape[1]
    st = stream if stream is not None else torch.cuda.current_stream()
    status = lib.seg_label_loss_noalloc(_ptr(out), _ptr(cls), _ptr(sil), sil.shape[0], out.shape[1], out.shape[0],
                                        int(bool(relu_mask)), _ptr(dz), _ptr(loss_out), c_void_p(st.cuda_stream))
    if status != SEG_OK:
        raise SegError(status, "seg_label_loss_noalloc")


def handoff_copy(producer, src, consumer, dst):
    """seg_handoff_copy: the stored response `src` (on the producer's device) into `dst` (same shape and
    dtype, on the consumer's device); the consumer's stream waits for the copy."""
    assert src.is_cuda and dst.is_cuda and src.is_contiguous() and dst.is_contiguous()
    assert src.shape == dst.shape and src.dtype == dst.dtype
    producer._check(producer.lib.seg_handoff_copy(producer.h, _ptr(src), consumer.h, _ptr(dst),
                                                  src.numel() * src.element_size()), "seg_handoff_copy")


def train_partitioned(segments, x, cls, batch, epochs):
    """The paper's training procedure (Section 2, two or more partitions): segment k is trained for
    epochs[k] passes on the stored response of segment k-1 (segment 0 on x) against its own
    intermediate labels - the last segment against the class labels - and only then is its response
    over the whole set computed and handed to segment k+1.  Returns the per-step losses of every
    segment (device tensors) and the last segment's input.  Marshalling only: every step runs in
    seg_train_epochs / seg_forward_dataset.

    Segments may live on different devices (Section 2.1: one partition per GPU, the only transfer being
    the previous partition's stored response, once): x and cls are on the first segment's device; the
    response of segment k is copied into the next segment's device by seg_handoff_copy, the class
    indices by torch, before that segment's first step."""
    import torch
    losses = []
    cur, cur_cls = x, cls
    for k, (seg, n_ep) in enumerate(zip(segments, epochs)):
        steps = n_ep * (-(-cur.shape[0] // batch))
        with torch.cuda.device(seg.device):
            l = torch.zeros(max(steps, 1), device="cuda")
        seg.train_epochs(cur, cur_cls, batch, n_ep, l)
        losses.append(l[:steps])
        if k + 1 < len(segments):
            nxt = segments[k + 1]
            resp = seg.forward_dataset(cur, batch)
            if nxt.device != seg.device:
                dst = nxt._empty(*resp.shape, dtype=resp.dtype)
                handoff_copy(seg, resp, nxt, dst)
                seg.stream.synchronize()             # resp may be released once the copy has run
                resp = dst
                cur_cls = cur_cls.to(f"cuda:{nxt.device}")
            cur = resp
    return losses, cur


def train_partitioned_ranks(seg, x, cls, batch, epochs, rank, world, n_samples=None):
    """The same procedure with one partition per process (one rank per GPU, torch.distributed already
    initialised; Section 2.1: each partition trains within its own GPU and the only transfer is the
    previous partition's stored response, once).  Rank k owns segment k (`seg`), trains it for `epochs`
    passes and sends its stored response to rank k + 1 as ONE point-to-point message; rank 0 reads x,
    later ranks receive their input (x is ignored there and may be None).  cls, the class indices, must
    be present on every rank (they are labels of the data set, not something a partition computes).
    There is no collective and nothing else crosses between ranks.  `seg` needs train_epochs(x, cls,
    batch, epochs, losses), forward_dataset(x, batch), widths and act_dtype, which Segment provides.
    Returns (per-step losses of this rank's segment, this rank's input)."""
    import torch
    import torch.distributed as dist
    n = int(cls.shape[0] if n_samples is None else n_samples)
    if rank == 0:
        cur = x
    else:
        cur = torch.empty(n, seg.widths[0], dtype=seg.act_dtype, device=cls.device)
        dist.recv(cur, src=rank - 1)                    # the one transfer into this partition
    steps = epochs * (-(-n // batch))
    losses = torch.zeros(max(steps, 1), dtype=torch.float32, device=cls.device)
    seg.train_epochs(cur, cls, batch, epochs, losses)
    if rank + 1 < world:
        resp = seg.forward_dataset(cur, batch)
        if resp.is_cuda:
            torch.cuda.current_stream(resp.device).synchronize()
            seg.stream.synchronize()                    # the response is complete before it leaves the device
        dist.send(resp.contiguous(), dst=rank + 1)
    return losses[:steps], cur


def recovery_step(left, right, x, cls, loss_out=None):
    """seg_recovery_step: one step of the paper's recovery phase (left trained through the frozen right)."""
    assert x.is_cuda and x.is_contiguous() and x.dtype == left.act_dtype and x.shape[1] == left.widths[0]
    assert cls.is_cuda and cls.is_contiguous() and cls.shape[0] == x.shape[0]
    left._check(left.lib.seg_recovery_step(left.h, right.h, _ptr(x), _ptr(cls), x.shape[0], _ptr(loss_out)),
                "seg_recovery_step")
    left.last_batch = right.last_batch = x.shape[0]


def predict(segments, x, batch):
    """The joined network (Section 2: the partitions are joined after training): class = argmax of the
    last segment's logits."""
    cur = x
    for seg in segments:
        cur = seg.forward_dataset(cur, batch)
    return cur.argmax(dim=1)


class Segment:
    """One network segment on the current CUDA device.  Tensors are torch CUDA tensors."""

    def __init__(self, widths, n_classes, is_final, *, precision="fp32", optimizer="sgd", lr=0.01,
                 momentum=0.9, beta1=0.9, beta2=0.999, eps=1e-8, max_batch=256, segment_id=0,
                 init_seed=2, last_relu=None, gemm_backend="auto", stream=None, device=None):
        import torch
        self._torch = torch
        if not torch.cuda.is_available():
            raise RuntimeError("Segment needs a CUDA device; there is no CPU path")
        self.lib = load()
        self.device = torch.cuda.current_device() if device is None else int(device)
        self.widths = [int(w) for w in widths]
        self.n_layers = len(self.widths) - 1
        self.n_classes, self.is_final, self.precision = int(n_classes), bool(is_final), precision
        self.max_batch = int(max_batch)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._warr = (c_int32 * len(self.widths))(*self.widths)
        cfg = seg_config(self.n_layers, self._warr, self.n_classes, int(self.is_final),
                         -1 if last_relu is None else int(bool(last_relu)), int(segment_id),
                         PRECISIONS[precision], OPTIMIZERS[optimizer], lr, momentum, beta1, beta2, eps,
                         self.max_batch, BACKENDS[gemm_backend], int(init_seed),
                         c_void_p(self.stream.cuda_stream))
        self.h = c_void_p()
        with torch.cuda.device(self.device):          # the handle lives on the device current at seg_create
            self._check(self.lib.seg_create(byref(cfg), byref(self.h)), "seg_create")
        self.act_dtype = torch.bfloat16 if precision == "bf16" else torch.float32
        self.out_dtype = torch.float32 if self.is_final else self.act_dtype
        self.last_batch = 0

    # -- plumbing -------------------------------------------------------------------------
    def _check(self, status, what=""):
        if status != SEG_OK:
            detail = what
            if self.h:
                err = self.lib.seg_last_error(self.h).decode()
                detail = f"{what}: {err}" if err else what
            raise SegError(status, detail)

    def _empty(self, *shape, dtype=None):
        with self._torch.cuda.device(self.device), self._torch.cuda.stream(self.stream):
            return self._torch.empty(*shape, dtype=dtype or self._torch.float32, device="cuda")

    def close(self):
        if getattr(self, "h", None):
            self.lib.seg_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the five calls -------------------------------------------------------------------------
    def gen_labels(self, seed, dist="uniform_kappa", kappa=10.0):
        self._check(self.lib.seg_gen_labels(self.h, int(seed), LABEL_DISTS[dist], float(kappa)), "seg_gen_labels")

    def train_step(self, x, cls, loss_out=None, y_out=None):
        batch = x.shape[0]
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.act_dtype and x.shape[1] == self.widths[0]
        assert cls.is_cuda and cls.is_contiguous() and cls.dtype == self._torch.int32 and cls.shape[0] == batch
        self._check(self.lib.seg_train_step(self.h, _ptr(x), _ptr(cls), batch, _ptr(loss_out), _ptr(y_out)),
                    "seg_train_step")
        self.last_batch = batch

    def train_step_label_input(self, sil_in, cls, loss_out=None):
        """seg_train_step_label_input: the sample's input is row cls[b] of the previous cut's label matrix."""
        assert sil_in.is_cuda and sil_in.is_contiguous() and sil_in.dtype == self._torch.float32
        assert sil_in.shape == (self.n_classes, self.widths[0]) and cls.is_cuda and cls.dtype == self._torch.int32
        self._check(self.lib.seg_train_step_label_input(self.h, _ptr(sil_in), _ptr(cls), cls.shape[0], _ptr(loss_out)),
                    "seg_train_step_label_input")
        self.last_batch = cls.shape[0]

    def train_step_host(self, x_host, cls_host):
        """x_host / cls_host: CPU tensors (pinned for speed).  Returns the loss as a float."""
        batch = x_host.shape[0]
        assert not x_host.is_cuda and x_host.is_contiguous() and x_host.dtype == self.act_dtype
        assert not cls_host.is_cuda and cls_host.dtype == self._torch.int32
        loss = c_float()
        self._check(self.lib.seg_train_step_host(self.h, c_void_p(x_host.data_ptr()),
                                                 c_void_p(cls_host.data_ptr()), batch, byref(loss)),
                    "seg_train_step_host")
        self.last_batch = batch
        return loss.value

    def train_step_host_async(self, x_host, cls_host, loss_host=None):
        """seg_train_step_host_async: pinned CPU tensors in, nothing waited for.  loss_host: a pinned
        float32 CPU tensor (one element) the step's loss is written to when the step has run."""
        batch = x_host.shape[0]
        assert not x_host.is_cuda and x_host.is_contiguous() and x_host.dtype == self.act_dtype
        assert not cls_host.is_cuda and cls_host.dtype == self._torch.int32
        lp = None if loss_host is None else c_void_p(loss_host.data_ptr())
        self._check(self.lib.seg_train_step_host_async(self.h, c_void_p(x_host.data_ptr()),
                                                       c_void_p(cls_host.data_ptr()), batch, lp),
                    "seg_train_step_host_async")
        self.last_batch = batch

    def forward(self, x, y=None):
        batch = x.shape[0]
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.act_dtype and x.shape[1] == self.widths[0]
        if y is None:
            y = self._empty(batch, self.widths[-1], dtype=self.out_dtype)
        self._check(self.lib.seg_forward(self.h, _ptr(x), batch, _ptr(y)), "seg_forward")
        self.last_batch = batch
        return y

    def train_epochs(self, x, cls, batch, epochs, losses=None):
        """seg_train_epochs: `epochs` passes over the resident data set in stored order (no shuffling)."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.act_dtype and x.shape[1] == self.widths[0]
        assert cls.is_cuda and cls.is_contiguous() and cls.dtype == self._torch.int32 and cls.shape[0] == x.shape[0]
        self._check(self.lib.seg_train_epochs(self.h, _ptr(x), _ptr(cls), x.shape[0], int(batch), int(epochs),
                                              _ptr(losses)), "seg_train_epochs")
        self.last_batch = x.shape[0] % batch or batch

    def forward_dataset(self, x, batch, y=None):
        """seg_forward_dataset: the segment's stored response over the whole set."""
        assert x.is_cuda and x.is_contiguous() and x.dtype == self.act_dtype and x.shape[1] == self.widths[0]
        if y is None:
            y = self._empty(x.shape[0], self.widths[-1], dtype=self.out_dtype)
        self._check(self.lib.seg_forward_dataset(self.h, _ptr(x), x.shape[0], int(batch), _ptr(y)),
                    "seg_forward_dataset")
        self.last_batch = x.shape[0] % batch or batch
        return y

    # -- inspection -------------------------------------------------------------------------
    def labels(self):
        t = self._empty(self.n_classes, self.widths[-1])
        self._check(self.lib.seg_get_labels(self.h, _ptr(t)), "seg_get_labels")
        return t

    def set_labels(self, t):
        assert t.is_cuda and t.is_contiguous() and t.dtype == self._torch.float32
        self._check(self.lib.seg_set_labels(self.h, _ptr(t)), "seg_set_labels")

    def _pair(self, fn, layer, *extra):
        w = self._empty(self.widths[layer + 1], self.widths[layer])
        b = self._empty(self.widths[layer + 1])
        self._check(fn(self.h, layer, *extra, _ptr(w), _ptr(b)), fn.__name__)
        return w, b

    def params(self, layer):
        return self._pair(self.lib.seg_get_params, layer)

    def grads(self, layer):
        return self._pair(self.lib.seg_get_grads, layer)

    def opt_state(self, layer, which):
        return self._pair(self.lib.seg_get_opt_state, layer, which)

    def set_params(self, layer, W, b):
        W = W.contiguous().float()
        b = b.contiguous().float()
        self._check(self.lib.seg_set_params(self.h, layer, _ptr(W), _ptr(b)), "seg_set_params")
        self.stream.synchronize()

    def set_opt_state(self, layer, which, sW, sb):
        sW = sW.contiguous().float()
        sb = sb.contiguous().float()
        self._check(self.lib.seg_set_opt_state(self.h, layer, which, _ptr(sW), _ptr(sb)), "seg_set_opt_state")
        self.stream.synchronize()

    def step_count(self):
        n = c_uint64()
        self._check(self.lib.seg_get_step(self.h, byref(n)), "seg_get_step")
        return n.value

    def set_step(self, t):
        self._check(self.lib.seg_set_step(self.h, int(t)), "seg_set_step")

    def activation(self, layer):
        t = self._empty(self.last_batch, self.widths[layer])
        self._check(self.lib.seg_get_activation(self.h, layer, _ptr(t)), "seg_get_activation")
        return t

    def mem_bytes(self):
        cur, peak = c_uint64(), c_uint64()
        self._check(self.lib.seg_mem_bytes(self.h, byref(cur), byref(peak)), "seg_mem_bytes")
        return cur.value, peak.value

    def launch_count(self):
        n = c_uint64()
        self._check(self.lib.seg_launch_count(self.h, byref(n)), "seg_launch_count")
        return n.value

    def product_launches(self):
        """seg_product_launches as a dict: launches per product-kernel family."""
        c = (c_uint64 * 5)()
        self._check(self.lib.seg_product_launches(self.h, c), "seg_product_launches")
        return dict(zip(PRODUCT_FAMILIES, (int(v) for v in c)))

    def poll(self):
        self._check(self.lib.seg_poll_status(self.h), "seg_poll_status")

    def selftest_bounded_wait(self, limit_ns):
        self._check(self.lib.seg_selftest_bounded_wait(self.h, int(limit_ns)), "seg_selftest_bounded_wait")

    def timer_start(self):
        self._check(self.lib.seg_timer_start(self.h))

    def timer_stop(self):
        self._check(self.lib.seg_timer_stop(self.h))

    def timer_ms(self):
        ms = c_float()
        self._check(self.lib.seg_timer_elapsed_ms(self.h, byref(ms)))
        return ms.value

    def profile(self, on):
        self._check(self.lib.seg_profile_enable(self.h, int(on)))

    def profile_read(self):
        out = {}
        for k, name in KERNEL_KINDS.items():
            n, ms = c_uint64(), c_float()
            self._check(self.lib.seg_profile_get(self.h, k, byref(n), byref(ms)))
            out[name] = (n.value, ms.value)
        return out
