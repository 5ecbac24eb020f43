"""ctypes binding of libpipemare.so: the same entry points as include/pipemare.h, argument marshalling only.

`Pipeline` and `FlatUpdate` are conveniences that allocate the caller-owned device
buffers as torch tensors, pack parameters into the flat arenas with the layout the
library reports, and pass raw pointers through.  No arithmetic of the method happens
here.
"""
import ctypes as C
import os

import numpy as np

PM_F32, PM_BF16 = 0, 1
PM_SGDM, PM_ADAM = 0, 1
PM_ACT_NONE, PM_ACT_RELU, PM_ACT_GELU = 0, 1, 2
PM_OP_LINEAR, PM_OP_EMBED, PM_OP_LAYERNORM, PM_OP_ATTENTION, PM_OP_SKIP_OUT, PM_OP_RESIDUAL = 0, 1, 2, 3, 4, 5
PM_OP_CROSS_ATTENTION = 6
PM_OPF_CAUSAL, PM_OPF_FROM_MEMORY, PM_OPF_SECOND_STREAM, PM_OPF_EMIT_MEMORY, PM_OPF_SKIP_TWO = 1, 2, 4, 8, 16
PM_LOSS_MSE, PM_LOSS_CE = 0, 1
PM_TICK_MAJOR, PM_MB_MAJOR = 0, 1
PM_ALIGN_ELEMS = 64

_ACT = {"none": PM_ACT_NONE, "relu": PM_ACT_RELU, "gelu": PM_ACT_GELU}
_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpipemare.so")


class pm_op_desc(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_in", C.c_int32), ("n_out", C.c_int32), ("act", C.c_int32),
                ("n_heads", C.c_int32), ("seq_len", C.c_int32), ("flags", C.c_int32)]


class pm_stage_desc(C.Structure):
    _fields_ = [("tau_fwd", C.c_int32), ("tau_bkwd", C.c_int32), ("n_ops", C.c_int32),
                ("ops", C.POINTER(pm_op_desc)), ("param_offset", C.c_uint64), ("param_count", C.c_uint64)]


class pm_config(C.Structure):
    _fields_ = [("n_stages", C.c_int32), ("microbatch", C.c_int32), ("compute_dtype", C.c_int32),
                ("optimizer", C.c_int32), ("loss", C.c_int32),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("t1_enable", C.c_int32), ("t1_K", C.c_int64), ("t2_enable", C.c_int32), ("t2_D", C.c_double),
                ("alpha_const", C.c_double), ("alpha_by_step", C.POINTER(C.c_double)), ("alpha_len", C.c_int64),
                ("loss_log_capacity", C.c_int64), ("loop_order", C.c_int32), ("entry_period", C.c_int32), ("n_micro", C.c_int32),
                ("recompute_segment", C.c_int32), ("fuse_update", C.c_int32),
                ("stochastic_tau_max", C.c_int32), ("materialize_backward", C.c_int32)]


class pm_arenas(C.Structure):
    _fields_ = [("w", C.c_void_p), ("m", C.c_void_p), ("s", C.c_void_p), ("delta", C.c_void_p),
                ("grad", C.c_void_p), ("w_lp", C.c_void_p), ("count", C.c_uint64)]


class PipeMareError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"{status}: {message}")
        self.status = status


_lib = None


def lib():
    """Load libpipemare.so (once).  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise PipeMareError("PM_ERR_NOLIB", f"{LIB_PATH} is missing; run paper_1910_05124_b200/build.py "
                                            "(or __graft_entry__.build()) first")
    L = C.CDLL(LIB_PATH)
    vp, u64p = C.c_void_p, C.POINTER(C.c_uint64)
    L.pm_status_string.restype = C.c_char_p
    L.pm_status_string.argtypes = [C.c_int]
    L.pm_last_error.restype = C.c_char_p
    L.pm_last_error.argtypes = [vp]
    L.pm_stage_param_count.argtypes = [C.POINTER(pm_op_desc), C.c_int32, u64p]
    L.pm_op_param_offsets.argtypes = [C.POINTER(pm_op_desc), C.c_int32, C.c_int32, u64p, u64p]
    L.pm_query_bytes.argtypes = [C.POINTER(pm_config), C.POINTER(pm_stage_desc), u64p, u64p, u64p]
    L.pm_set_delays.argtypes = [C.c_void_p, C.POINTER(C.c_int32)]
    L.pm_init_stages.argtypes = [C.POINTER(vp), C.POINTER(pm_config), C.POINTER(pm_stage_desc), C.POINTER(pm_arenas),
                                 vp, C.c_uint64, vp, C.c_uint64, vp]
    L.pm_set_warmup.argtypes = [vp, C.c_int64]
    L.pm_forward.argtypes = [vp, vp, vp]
    L.pm_backward.argtypes = [vp]
    L.pm_update.argtypes = [vp]
    L.pm_step.argtypes = [vp, vp, vp]
    L.pm_get_bookkeeping.argtypes = [vp, C.c_int32, C.POINTER(C.c_int64)]
    L.pm_get_losses.argtypes = [vp, C.POINTER(C.c_float), C.c_int64, C.c_int64]
    L.pm_selftest_wait_timeout.argtypes = [vp, C.c_int64]
    L.pm_launch_count.argtypes = [vp]
    L.pm_launch_count.restype = C.c_uint64
    L.pm_profile_enable.argtypes = [vp, C.c_int32]
    L.pm_profile_read.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
    L.pm_destroy.argtypes = [vp]
    L.pm_destroy.restype = None
    L.pm_update_flat_workspace_bytes.argtypes = [C.c_int32]
    L.pm_update_flat_workspace_bytes.restype = C.c_uint64
    L.pm_update_flat.argtypes = [C.POINTER(pm_arenas), u64p, u64p, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                 C.c_int32, C.POINTER(pm_config), C.c_int64, vp, C.c_uint64, vp]
    L.pm_update_flat_static.argtypes = [C.POINTER(pm_arenas), u64p, u64p, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                        C.c_int32, C.POINTER(pm_config), C.c_int64, vp]
    L.pm_update_flat_static_max_stages.restype = C.c_int32
    L.pm_update_flat_static_last_error.restype = C.c_char_p
    _lib = L
    return L


def _check(status, ctx=None):
    if status != 0:
        L = lib()
        raise PipeMareError(L.pm_status_string(status).decode(), L.pm_last_error(ctx).decode())


def make_config(*, n_stages, microbatch, compute, optimizer, alpha, beta1=0.9, beta2=0.98, eps=1e-8,
                t1=True, K=1, t2=True, D=0.5, alpha_by_step=None, loss_log_capacity=0, loss=PM_LOSS_MSE,
                loop_order=PM_TICK_MAJOR, n_micro=1, entry_period=0, recompute_segment=0, fuse_update=0, stochastic_tau_max=0, materialize_backward=0):
    cfg = pm_config()
    cfg.n_stages, cfg.microbatch = n_stages, microbatch
    cfg.compute_dtype = PM_BF16 if compute in ("bf16", PM_BF16) and compute != 0 else PM_F32
    cfg.optimizer = PM_ADAM if optimizer in ("adam", PM_ADAM) and optimizer != 0 else PM_SGDM
    cfg.loss = loss
    cfg.beta1, cfg.beta2, cfg.eps = beta1, beta2, eps
    cfg.t1_enable, cfg.t1_K = int(bool(t1)), int(K)
    cfg.t2_enable, cfg.t2_D = int(bool(t2)), float(D)
    cfg.alpha_const = float(alpha)
    keep = None
    if alpha_by_step is not None:
        keep = (C.c_double * len(alpha_by_step))(*alpha_by_step)
        cfg.alpha_by_step = C.cast(keep, C.POINTER(C.c_double))
        cfg.alpha_len = len(alpha_by_step)
    cfg.loss_log_capacity = loss_log_capacity
    cfg.loop_order = PM_MB_MAJOR if loop_order in ("mb_major", PM_MB_MAJOR) and loop_order != 0 else PM_TICK_MAJOR
    cfg.n_micro = int(n_micro)
    cfg.recompute_segment = int(recompute_segment)
    cfg.fuse_update = int(bool(fuse_update))
    cfg.stochastic_tau_max = int(stochastic_tau_max)
    cfg.materialize_backward = int(bool(materialize_backward))
    cfg.entry_period = int(entry_period)
    return cfg, keep


def _ops_array(specs):
    """ctypes op array of an MLP stage (a list of Linear specs)."""
    return _ops_from_dicts([dict(kind=PM_OP_LINEAR, n_in=sp.n_in, n_out=sp.n_out, act=_ACT[sp.act]) for sp in specs])


def _ops_from_dicts(ops):
    arr = (pm_op_desc * len(ops))()
    for j, o in enumerate(ops):
        arr[j].kind, arr[j].n_in, arr[j].n_out = o["kind"], o.get("n_in", 0), o.get("n_out", 0)
        arr[j].act, arr[j].n_heads, arr[j].seq_len = o.get("act", 0), o.get("n_heads", 0), o.get("seq_len", 0)
        arr[j].flags = o.get("flags", 0)
    return arr


def stage_ops(wl, p):
    """Op list of stage p and, per parameter tensor in the workload's order, (op index, slot, shape)."""
    if getattr(wl, "kind", "mlp") == "encoder":
        sp = wl.stage_specs[p]
        ops, tensors = [], []
        if sp.pre in ("embed", "embed_dec"):
            ops.append(dict(kind=PM_OP_EMBED, n_in=wl.vocab, n_out=wl.d_model, seq_len=wl.seq_len,
                            flags=PM_OPF_SECOND_STREAM if sp.pre == "embed_dec" else 0))
            tensors.append((0, 0, (wl.vocab, wl.d_model)))
        elif sp.pre == "ln":
            ops.append(dict(kind=PM_OP_LAYERNORM, n_in=sp.n_in, n_out=sp.n_in,
                            flags=PM_OPF_FROM_MEMORY if getattr(sp, "src", "main") == "memory" else 0))
            tensors += [(0, 0, (sp.n_in,)), (0, 1, (sp.n_in,))]
        li = len(ops)
        ops.append(dict(kind=PM_OP_LINEAR, n_in=sp.n_in, n_out=sp.n_out, act=_ACT[sp.act]))
        tensors += [(li, 0, (sp.n_out, sp.n_in)), (li, 1, (sp.n_out,))]
        if sp.post == "attention":
            ops.append(dict(kind=PM_OP_ATTENTION, n_in=sp.n_out, n_out=sp.n_out // 3, n_heads=wl.n_heads, seq_len=wl.seq_len,
                            flags=PM_OPF_CAUSAL if getattr(sp, "causal", False) else 0))
        elif sp.post == "cross_attention":
            ops.append(dict(kind=PM_OP_CROSS_ATTENTION, n_in=sp.n_out, n_out=sp.n_out // 2, n_heads=wl.n_heads, seq_len=wl.seq_len))
        elif sp.post == "skip_out":
            ops.append(dict(kind=PM_OP_SKIP_OUT, flags=PM_OPF_SKIP_TWO if getattr(sp, "skip_hop", 1) == 2 else 0))
        elif sp.post == "residual":
            ops.append(dict(kind=PM_OP_RESIDUAL, flags=PM_OPF_EMIT_MEMORY if getattr(sp, "emit_memory", False) else 0))
        return ops, tensors
    ops, tensors = [], []
    for j, sp in enumerate(wl.stages[p]):
        ops.append(dict(kind=PM_OP_LINEAR, n_in=sp.n_in, n_out=sp.n_out, act=_ACT[sp.act]))
        tensors += [(j, 0, (sp.n_out, sp.n_in)), (j, 1, (sp.n_out,))]
    return ops, tensors


def ops_layout(arr, n_ops, tensors):
    """(padded element count of the stage, offset of each parameter tensor), as the library lays it out."""
    L = lib()
    cnt = C.c_uint64()
    _check(L.pm_stage_param_count(arr, n_ops, C.byref(cnt)))
    offs = []
    for (op, slot, shape) in tensors:
        a, b = C.c_uint64(), C.c_uint64()
        _check(L.pm_op_param_offsets(arr, n_ops, op, C.byref(a), C.byref(b)))
        offs.append(a.value if slot == 0 else b.value)
    return cnt.value, offs


def stage_layout(specs):
    """(padded element count, [(w_off, b_off) per op]) of an MLP stage, as the library lays it out."""
    arr = _ops_array(specs)
    tensors = [t for j, sp in enumerate(specs) for t in ((j, 0, None), (j, 1, None))]
    cnt, offs = ops_layout(arr, len(specs), tensors)
    return cnt, [(offs[2 * j], offs[2 * j + 1]) for j in range(len(specs))]


class Pipeline:
    """Owns the device buffers of one pipeline context and forwards calls to the C ABI.

    wl: a workload description with fields stages (lists of objects with n_in, n_out, act),
    tau_fwd, tau_bkwd, microbatch, compute, optimizer, alpha, beta1, beta2, eps, t1, K, t2, D.
    params0: per stage a list of (W[out,in], b[out]) float32 numpy arrays.
    """

    def __init__(self, wl, params0, device="cuda:0", stream=None, loss_log_capacity=0, loop_order=PM_TICK_MAJOR, n_micro=1, entry_period=0,
                 recompute_segment=0, fuse_update=0, stochastic_tau_max=0, materialize_backward=0):
        import torch
        self.torch = torch
        self.wl = wl
        self.L = lib()
        self.device = torch.device(device)
        P = wl.n_stages
        self.P = P
        self.is_encoder = getattr(wl, "kind", "mlp") == "encoder"
        self._op_dicts, self._tensors, self._ops, self.layout = [], [], [], []
        for p in range(P):
            ops, tensors = stage_ops(wl, p)
            arr = _ops_from_dicts(ops)
            self._op_dicts.append(ops)
            self._tensors.append(tensors)
            self._ops.append(arr)
            self.layout.append(ops_layout(arr, len(ops), tensors))
        self.stage_desc = (pm_stage_desc * P)()
        off = 0
        for p in range(P):
            d = self.stage_desc[p]
            d.tau_fwd, d.tau_bkwd, d.n_ops = wl.tau_fwd[p], wl.tau_bkwd[p], len(self._op_dicts[p])
            d.ops = C.cast(self._ops[p], C.POINTER(pm_op_desc))
            d.param_offset, d.param_count = off, self.layout[p][0]
            off += self.layout[p][0]
        self.total = off
        self.cfg, self._alpha_keep = make_config(
            n_stages=P, microbatch=wl.microbatch, compute=wl.compute, optimizer=wl.optimizer, alpha=wl.alpha,
            beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, t1=wl.t1, K=wl.K, t2=wl.t2, D=wl.D,
            loss_log_capacity=loss_log_capacity, loss=PM_LOSS_CE if self.is_encoder else PM_LOSS_MSE,
            loop_order=loop_order, n_micro=n_micro, entry_period=entry_period, recompute_segment=recompute_segment,
            fuse_update=fuse_update, stochastic_tau_max=stochastic_tau_max,
            materialize_backward=materialize_backward)
        self.mb_major = self.cfg.loop_order == PM_MB_MAJOR
        sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
        _check(self.L.pm_query_bytes(C.byref(self.cfg), self.stage_desc, C.byref(sb), C.byref(rb), C.byref(wb)))
        self.state_bytes, self.ring_bytes, self.workspace_bytes = sb.value, rb.value, wb.value
        dev = self.device
        f32 = dict(dtype=torch.float32, device=dev)
        self.w = torch.zeros(self.total, **f32)
        self.m = torch.zeros(self.total, **f32)
        self.delta = torch.zeros(self.total, **f32)
        self.grad = torch.zeros(self.total, **f32)
        self.s = torch.zeros(self.total, **f32) if wl.optimizer == "adam" else None
        flat = np.zeros(self.total, dtype=np.float32)
        for p in range(P):
            base = self.stage_desc[p].param_offset
            tensors = params0[p]
            if not self.is_encoder:                       # MLP stages come as (W, b) pairs
                tensors = [a for pair in tensors for a in pair]
            for a, o in zip(tensors, self.layout[p][1]):
                a = np.asarray(a, dtype=np.float32)
                flat[base + o: base + o + a.size] = a.ravel()
        self.w.copy_(torch.from_numpy(flat))
        self.w_lp = self.w.to(torch.bfloat16) if wl.compute == "bf16" else None
        self.ring = torch.empty(max(self.ring_bytes, 256), dtype=torch.uint8, device=dev)
        self.workspace = torch.empty(max(self.workspace_bytes, 256), dtype=torch.uint8, device=dev)
        self.stream = stream if stream is not None else torch.cuda.current_stream(dev)
        self.arenas = pm_arenas(self.w.data_ptr(), self.m.data_ptr(), self.s.data_ptr() if self.s is not None else None,
                                self.delta.data_ptr(), self.grad.data_ptr(),
                                self.w_lp.data_ptr() if self.w_lp is not None else None, self.total)
        self.ctx = C.c_void_p()
        torch.cuda.synchronize(dev)
        _check(self.L.pm_init_stages(C.byref(self.ctx), C.byref(self.cfg), self.stage_desc, C.byref(self.arenas),
                                     self.ring.data_ptr(), self.ring.numel(), self.workspace.data_ptr(),
                                     self.workspace.numel(), C.c_void_p(self.stream.cuda_stream)))

    # -- the C entry points, same names -------------------------------------------------------
    def _ptr(self, t):
        return None if t is None else C.c_void_p(t.data_ptr())

    def pm_set_delays(self, delays):
        arr = (C.c_int32 * self.P)(*[int(d) for d in delays])
        _check(self.L.pm_set_delays(self.ctx, arr), self.ctx)

    def pm_set_warmup(self, n_microbatches):
        _check(self.L.pm_set_warmup(self.ctx, int(n_microbatches)), self.ctx)

    def pm_forward(self, inputs=None, targets=None):
        _check(self.L.pm_forward(self.ctx, self._ptr(inputs), self._ptr(targets)), self.ctx)

    def pm_backward(self):
        _check(self.L.pm_backward(self.ctx), self.ctx)

    def pm_update(self):
        _check(self.L.pm_update(self.ctx), self.ctx)

    def pm_step(self, inputs=None, targets=None):
        _check(self.L.pm_step(self.ctx, self._ptr(inputs), self._ptr(targets)), self.ctx)

    def pm_get_bookkeeping(self, stage):
        out = (C.c_int64 * 8)()
        _check(self.L.pm_get_bookkeeping(self.ctx, stage, out), self.ctx)
        return list(out)

    def pm_get_losses(self, first_mb, n):
        out = (C.c_float * n)()
        _check(self.L.pm_get_losses(self.ctx, out, first_mb, n), self.ctx)
        return np.array(out[:], dtype=np.float32)

    def pm_selftest_wait_timeout(self, limit_cycles):
        """Returns the status name the library reports after a bounded device wait expired (PM_ERR_TIMEOUT)."""
        st = self.L.pm_selftest_wait_timeout(self.ctx, int(limit_cycles))
        return self.L.pm_status_string(st).decode(), self.L.pm_last_error(self.ctx).decode()

    def pm_launch_count(self):
        return int(self.L.pm_launch_count(self.ctx))

    PROF_CLASSES = ["schedule", "ingest", "pre_fwd", "gemm_fwd", "attn_fwd", "post_fwd", "loss", "attn_bwd", "act_bwd",
                    "wgrad", "dgrad", "pre_bwd", "update"]

    def pm_profile_enable(self, on=True):
        _check(self.L.pm_profile_enable(self.ctx, int(bool(on))), self.ctx)

    def pm_profile_read(self):
        """{class name: (milliseconds, launches)} since the last read."""
        n = len(self.PROF_CLASSES)
        ms, cnt = (C.c_float * n)(), (C.c_int64 * n)()
        _check(self.L.pm_profile_read(self.ctx, ms, cnt), self.ctx)
        return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(self.PROF_CLASSES)}

    # -- marshalling helpers --------------------------------------------------------------------
    def unpack(self, flat_tensor):
        """Split a flat arena (device tensor) into per-stage parameter tensors (numpy): (W, b) pairs for MLP
        stages, the list [table] [gain, bias] W b for encoder stages."""
        flat = flat_tensor.detach().float().cpu().numpy()
        out = []
        for p in range(self.P):
            base = self.stage_desc[p].param_offset
            tensors = []
            for (op, slot, shape), o in zip(self._tensors[p], self.layout[p][1]):
                n = int(np.prod(shape))
                tensors.append(flat[base + o: base + o + n].reshape(shape).copy())
            if not self.is_encoder:
                tensors = [(tensors[2 * j], tensors[2 * j + 1]) for j in range(len(tensors) // 2)]
            out.append(tensors)
        return out

    def close(self):
        if self.ctx:
            self.L.pm_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class FlatUpdate:
    """Marshals pm_update_flat: holds the host tables and the device workspace for one stage split."""

    def __init__(self, offsets, counts, tau_fwd, tau_bkwd, *, optimizer, alpha, beta1=0.9, beta2=0.98, eps=1e-8,
                 t1=True, K=1, t2=True, D=0.5, device="cuda:0"):
        import torch
        self.torch = torch
        self.L = lib()
        P = len(offsets)
        self.P = P
        self.offsets = (C.c_uint64 * P)(*offsets)
        self.counts = (C.c_uint64 * P)(*counts)
        self.tau_fwd = (C.c_int32 * P)(*tau_fwd)
        self.tau_bkwd = (C.c_int32 * P)(*tau_bkwd)
        self.cfg, self._keep = make_config(n_stages=P, microbatch=1, compute="f32", optimizer=optimizer, alpha=alpha,
                                           beta1=beta1, beta2=beta2, eps=eps, t1=t1, K=K, t2=t2, D=D)
        self.ws_bytes = self.L.pm_update_flat_workspace_bytes(P)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=device)

    def pm_update_flat(self, w, m, s, delta, grad, w_lp, k, stream=None):
        torch = self.torch
        st = stream if stream is not None else torch.cuda.current_stream(w.device)
        ar = pm_arenas(w.data_ptr(), m.data_ptr(), s.data_ptr() if s is not None else None, delta.data_ptr(),
                       grad.data_ptr(), w_lp.data_ptr() if w_lp is not None else None, w.numel())
        _check(self.L.pm_update_flat(C.byref(ar), self.offsets, self.counts, self.tau_fwd, self.tau_bkwd, self.P,
                                     C.byref(self.cfg), k, self.workspace.data_ptr(), self.ws_bytes,
                                     C.c_void_p(st.cuda_stream)))

    def pm_update_flat_static(self, w, m, s, delta, grad, w_lp, k, stream=None):
        """Same update through the entry point that needs no device workspace: for callers that are not
        allowed to allocate on the device (the stage table sits in a fixed array inside the library)."""
        torch = self.torch
        st = stream if stream is not None else torch.cuda.current_stream(w.device)
        ar = pm_arenas(w.data_ptr(), m.data_ptr(), s.data_ptr() if s is not None else None, delta.data_ptr(),
                       grad.data_ptr(), w_lp.data_ptr() if w_lp is not None else None, w.numel())
        status = self.L.pm_update_flat_static(C.byref(ar), self.offsets, self.counts, self.tau_fwd, self.tau_bkwd,
                                              self.P, C.byref(self.cfg), k, C.c_void_p(st.cuda_stream))
        if status != 0:
            raise PipeMareError(self.L.pm_status_string(status).decode(),
                                self.L.pm_update_flat_static_last_error().decode())
