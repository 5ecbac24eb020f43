"""The C-ABI library loads on a machine without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built_lib():
    from paper_1910_05124_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "pipemare.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pm_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_required_entry_points():
    syms = declared_symbols()
    for name in ("pm_init_stages", "pm_forward", "pm_backward", "pm_update", "pm_step", "pm_update_flat",
                 "pm_query_bytes", "pm_get_bookkeeping", "pm_get_losses", "pm_destroy"):
        assert name in syms


def test_library_exports_every_declared_symbol(built_lib):
    for name in declared_symbols():
        assert hasattr(built_lib, name), name


def test_layout_arithmetic_needs_no_gpu(built_lib):
    import pm_inputs as I
    from paper_1910_05124_b200 import binding
    cnt, offs = binding.stage_layout(I.cfg3().stages[0])
    assert cnt == 2 * (1024 * 1024 + 1024)
    assert offs == [(0, 1024 * 1024), (1024 * 1024 + 1024, 2 * 1024 * 1024 + 1024)]
    cnt, offs = binding.stage_layout([I.LinearSpec(40, 24, "relu")])
    assert offs == [(0, 960)] and cnt == 960 + 64          # W padded to 960 (=15*64), b padded to 64


def test_query_bytes_and_state_copies_ratio(built_lib):
    # PipeMare adds one weight-sized accumulator: 4/3 of the SGD-momentum state, 5/4 of Adam's
    # (weight + optimiser memory relative to the synchronous baseline, Table 2 / Section 4.2)
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    wl = I.cfg1()
    for opt, ratio in (("sgdm", 4 / 3), ("adam", 5 / 4)):
        wl.optimizer = opt
        P = len(wl.stages)
        ops = [B._ops_array(st) for st in wl.stages]
        sd = (B.pm_stage_desc * P)()
        off = 0
        for p in range(P):
            cnt, _ = B.stage_layout(wl.stages[p])
            sd[p].tau_fwd, sd[p].tau_bkwd, sd[p].n_ops = wl.tau_fwd[p], 0, len(wl.stages[p])
            sd[p].ops = C.cast(ops[p], C.POINTER(B.pm_op_desc))
            sd[p].param_offset, sd[p].param_count = off, cnt
            off += cnt
        cfg, _ = B.make_config(n_stages=P, microbatch=32, compute="f32", optimizer=opt, alpha=0.01, K=32)
        sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
        assert B.lib().pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
        # state copies: weight, gradient, optimiser state (the synchronous baseline) plus delta
        copies = sb.value / (off * 4)
        baseline = 3 if opt == "sgdm" else 4            # w, g, v   |   w, g, m, s
        assert copies == baseline + 1
        assert copies / baseline == pytest.approx(ratio, rel=1e-12)
        # ring: (tau+2) input slots per stage; a ReLU's mask is read from the next stage's stashed input, which costs
        # that stage one more slot instead of (tau+1) pre-activation slots; only the last stage keeps pre-activations
        slots = sum(t + 2 for t in wl.tau_fwd) + (P - 1) + (wl.tau_fwd[-1] + 1)
        assert rb.value == slots * 32 * 256 * 4


def test_bad_arguments_are_rejected_without_a_gpu(built_lib):
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    L = B.lib()
    wl = I.cfg1()
    P = len(wl.stages)
    ops = [B._ops_array(st) for st in wl.stages]
    sd = (B.pm_stage_desc * P)()
    off = 0
    for p in range(P):
        cnt, _ = B.stage_layout(wl.stages[p])
        sd[p].tau_fwd, sd[p].tau_bkwd, sd[p].n_ops = wl.tau_fwd[p], 0, 1
        sd[p].ops = C.cast(ops[p], C.POINTER(B.pm_op_desc))
        sd[p].param_offset, sd[p].param_count = off, cnt
        off += cnt
    cfg, _ = B.make_config(n_stages=P, microbatch=32, compute="f32", optimizer="sgdm", alpha=0.01, K=32)
    sb = C.c_uint64()
    sd[1].tau_fwd = 4                                    # not 2(P-i)+1
    st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), None, None)
    assert L.pm_status_string(st) == b"PM_ERR_UNSUPPORTED"
    assert b"tau_fwd" in L.pm_last_error(None)
    sd[1].tau_fwd = 5
    ops[2][0].n_in = 128                                 # breaks the chain 256 -> 128
    st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), None, None)
    assert L.pm_status_string(st) == b"PM_ERR_SHAPE"
    assert L.pm_status_string(L.pm_forward(None, None, None)) == b"PM_ERR_INVALID_ARG"


def _describe(wl, mutate=None):
    """Stage descriptors of a Transformer workload as the binding builds them; mutate(p, ops) may edit a stage's op list."""
    import ctypes as C
    from paper_1910_05124_b200 import binding as B
    P = wl.n_stages
    sd = (B.pm_stage_desc * P)()
    keep, off = [], 0
    for p in range(P):
        ops, tensors = B.stage_ops(wl, p)
        if mutate:
            mutate(p, ops)
        arr = B._ops_from_dicts(ops)
        keep.append(arr)
        cnt, _ = B.ops_layout(arr, len(ops), tensors)
        sd[p].tau_fwd, sd[p].tau_bkwd, sd[p].n_ops = wl.tau_fwd[p], 0, len(ops)
        sd[p].ops = C.cast(arr, C.POINTER(B.pm_op_desc))
        sd[p].param_offset, sd[p].param_count = off, cnt
        off += cnt
    cfg, _ = B.make_config(n_stages=P, microbatch=wl.microbatch, compute=wl.compute, optimizer=wl.optimizer, alpha=wl.alpha,
                           beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, K=wl.K, D=wl.D, loss=B.PM_LOSS_CE)
    return cfg, sd, keep


def test_encoder_decoder_layout_and_its_checks(built_lib):
    """Footprints of the encoder-decoder workloads (host arithmetic only) and the chaining rules of their stages."""
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    L = B.lib()

    def query(wl, mutate=None):
        cfg, sd, keep = _describe(wl, mutate)
        sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
        st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))
        return L.pm_status_string(st), L.pm_last_error(None), sb.value, rb.value, wb.value

    # config 5 as given (133 stages, sequences of 256 tokens) is laid out, but its rings do not fit one GPU
    st, _, sb, rb, wb = query(I.cfg5())
    assert st == b"PM_OK" and rb > 400e9
    # beyond 128 tokens attention exists for 256 tokens, bf16 and heads of width 64 only
    st, msg = query(I.cfg5_small(compute="f32", d_model=128, n_heads=2, seq_len=256, batch=1))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"beyond 128 tokens" in msg
    st, msg = query(I.cfg5_small(compute="bf16", d_model=128, n_heads=2, seq_len=512, batch=1))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"beyond 128 tokens" in msg
    st, msg = query(I.cfg5_small(compute="bf16", d_model=128, n_heads=4, seq_len=256, batch=1))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"beyond 128 tokens" in msg
    assert query(I.cfg5_small(compute="bf16", d_model=128, n_heads=2, seq_len=256, batch=1))[0] == b"PM_OK"
    # its 12 + 12 layers do not fit one GPU in the tick-major stash plan; the 7 + 7 layer cut does, 8 + 8 does not
    st, _, sb, rb, wb = query(I.cfg5_cut(12, 12))
    assert st == b"PM_OK" and rb > 400e9 and sb < 12e9
    st, _, sb, rb, wb = query(I.cfg5_cut())
    assert st == b"PM_OK" and 145e9 < rb < 155e9 and sb + rb + wb < 170e9
    st, _, sb, rb, wb = query(I.cfg5_cut(8, 8))
    assert st == b"PM_OK" and sb + rb + wb > 200e9
    st, _, sb, rb, wb = query(I.cfg5_cut(4, 4))
    assert st == b"PM_OK" and 45e9 < rb < 55e9 and sb + rb + wb < 70e9
    small = I.cfg5_small()
    assert query(small)[0] == b"PM_OK"
    dec0 = [i for i, s in enumerate(small.stage_specs) if s.pre == "embed_dec"][0]

    def drop_flag(stage, kind, flag):
        def m(p, ops):
            if p == stage:
                for o in ops:
                    if o["kind"] == kind:
                        o["flags"] = o.get("flags", 0) & ~flag
        return m
    # the decoder's embedding without the second-stream flag, the memory stage without its flag, a two-stage skip
    # declared as a one-stage skip, a cross-attention stage whose LayerNorm reads the main stream
    st, msg = query(small, drop_flag(dec0, B.PM_OP_EMBED, B.PM_OPF_SECOND_STREAM))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"EMBED" in msg
    st, msg = query(small, drop_flag(dec0 - 1, B.PM_OP_RESIDUAL, B.PM_OPF_EMIT_MEMORY))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"memory" in msg
    st, msg = query(small, drop_flag(dec0 + 2, B.PM_OP_SKIP_OUT, B.PM_OPF_SKIP_TWO))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"RESIDUAL" in msg
    st, msg = query(small, drop_flag(dec0 + 3, B.PM_OP_LAYERNORM, B.PM_OPF_FROM_MEMORY))[:2]
    assert st == b"PM_ERR_UNSUPPORTED" and b"CROSS_ATTENTION" in msg


def test_microbatch_major_footprint_of_config5(built_lib):
    """The queue of weight versions: (tau_i + 1) bf16 copies of every stage's slice plus fp32 copies of its biases and
    LayerNorm parameters, and activations of one microbatch.  Config 5 as configured then fits one 180 GB GPU, which
    its tick-major rings (more than 400 GB) do not."""
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    L = B.lib()
    wl = I.cfg5()
    cfg, sd, keep = _describe(wl)
    cfg.loop_order = B.PM_MB_MAJOR
    sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    P = wl.n_stages
    queue = sum((wl.tau_fwd[p] + 1) * sd[p].param_count * 2 for p in range(P))     # the bf16 slices alone
    assert queue < rb.value < queue + 8e9                        # plus fp32 small tensors and one microbatch of activations
    assert 125e9 < rb.value < 140e9 and sb.value + rb.value + wb.value < 170e9
    # any forward delays are accepted in this order, a backward delay is not
    sd[3].tau_fwd = 0
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    sd[3].tau_bkwd = 1
    st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))
    assert L.pm_status_string(st) == b"PM_ERR_UNSUPPORTED"
    # ... unless it equals the forward delay in every stage (weight stashing): the same queues, nothing more to store
    sd[3].tau_fwd, sd[3].tau_bkwd = wl.tau_fwd[3], 0
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    queues = rb.value
    for p in range(P):
        sd[p].tau_bkwd = sd[p].tau_fwd
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0 and rb.value == queues
    sd[5].tau_bkwd = 0                                            # a mixture of the two patterns is not a mode
    st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))
    assert L.pm_status_string(st) == b"PM_ERR_UNSUPPORTED"
    for p in range(P):
        sd[p].tau_bkwd = 0
    cfg.loop_order = 7
    assert L.pm_status_string(L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))) == b"PM_ERR_INVALID_ARG"


def test_recompute_and_fused_update_options_are_checked_without_a_gpu(built_lib):
    """PipeMare Recompute: the queue of T2-corrected recompute weights is counted by pm_query_bytes (tau_recomp + 1 slots
    of every stage outside the last segment, tau_recomp = ceil-free 2(S - j) + 1 for one microbatch per update), and
    the options' preconditions are reported as PM_ERR_UNSUPPORTED."""
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    L = B.lib()
    wl = I.cfg5()
    P, S = wl.n_stages, 12
    cfg, sd, keep = _describe(wl)
    cfg.loop_order = B.PM_MB_MAJOR
    sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    plain = rb.value
    cfg.recompute_segment = S
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    last = (P - 1) // S * S                                   # first stage of the last segment: nothing is recomputed from there on
    extra = sum((2 * (min(P, (p // S + 1) * S) - 1 - p) + 1 + 1) * sd[p].param_count * 2 for p in range(last))
    assert extra < rb.value - plain < extra * 1.01            # plus the fp32 copies of biases and LayerNorm parameters
    cfg.recompute_segment = P                                 # one segment: the forward pass itself
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0 and rb.value == plain
    cfg.recompute_segment = -1
    assert L.pm_status_string(L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))) == b"PM_ERR_INVALID_ARG"
    cfg.recompute_segment = S
    cfg.loop_order = B.PM_TICK_MAJOR
    sd_t = sd                                                 # Table 1's delays: the tick schedule accepts them, but not the option
    assert L.pm_status_string(L.pm_query_bytes(C.byref(cfg), sd_t, C.byref(sb), C.byref(rb), C.byref(wb))) == b"PM_ERR_UNSUPPORTED"
    # the update in the weight-gradient epilogue: bf16, one Linear per stage, one microbatch per update, no recomputation
    cfg.loop_order, cfg.recompute_segment, cfg.fuse_update = B.PM_MB_MAJOR, 0, 1
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    for field, value in (("recompute_segment", S), ("n_micro", 2), ("compute_dtype", B.PM_F32)):
        old = getattr(cfg, field)
        setattr(cfg, field, value)
        st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))
        assert L.pm_status_string(st) == b"PM_ERR_UNSUPPORTED", field
        setattr(cfg, field, old)


def test_stochastic_delay_model_footprint_and_checks_without_a_gpu(built_lib):
    """Appendix E's model keeps the gradients of the last tau_max + 1 microbatches (copies of the grad arena) and one weight
    version per stage; its preconditions are reported as PM_ERR_UNSUPPORTED."""
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    L = B.lib()
    wl = I.cfg4()
    cfg, sd, keep = _describe(wl)
    cfg.loop_order = B.PM_MB_MAJOR
    sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
    total = sum(sd[p].param_count for p in range(wl.n_stages))
    sizes = {}
    for tmax in (1, 5):
        cfg.stochastic_tau_max = tmax
        assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
        sizes[tmax] = rb.value
    assert sizes[5] - sizes[1] == 4 * total * 4
    cfg.stochastic_tau_max = 0
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    assert rb.value > sizes[1] - 2 * total * 4                # without the model the stages queue tau_i + 1 weight versions instead
    cfg.stochastic_tau_max = 3
    for field, value in (("loop_order", B.PM_TICK_MAJOR), ("n_micro", 2), ("recompute_segment", 5), ("fuse_update", 1)):
        old = getattr(cfg, field)
        setattr(cfg, field, value)
        st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))
        assert L.pm_status_string(st) == b"PM_ERR_UNSUPPORTED", field
        setattr(cfg, field, old)
    cfg.stochastic_tau_max = -2
    assert L.pm_status_string(L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))) == b"PM_ERR_INVALID_ARG"


def test_materialize_backward_footprint_and_checks_without_a_gpu(built_lib):
    """The option keeps one more operand-type copy of every stage that has a delay gap (config 5: all of them) and is
    refused outside microbatch-major order or together with the options it does not combine with."""
    import ctypes as C
    import pm_inputs as I
    from paper_1910_05124_b200 import binding as B
    L = B.lib()
    wl = I.cfg5()
    cfg, sd, keep = _describe(wl)
    cfg.loop_order = B.PM_MB_MAJOR
    sb, rb, wb = C.c_uint64(), C.c_uint64(), C.c_uint64()
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    plain = rb.value
    cfg.materialize_backward = 1
    assert L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb)) == 0
    copy = sum(sd[p].param_count * 2 for p in range(wl.n_stages))
    assert copy <= rb.value - plain < copy * 1.01
    for field, value in (("loop_order", B.PM_TICK_MAJOR), ("recompute_segment", 12), ("stochastic_tau_max", 3), ("fuse_update", 1)):
        old = getattr(cfg, field)
        setattr(cfg, field, value)
        st = L.pm_query_bytes(C.byref(cfg), sd, C.byref(sb), C.byref(rb), C.byref(wb))
        assert L.pm_status_string(st) == b"PM_ERR_UNSUPPORTED", field
        setattr(cfg, field, old)


def test_flat_update_argument_checks_need_no_gpu(built_lib):
    """pm_update_flat / pm_update_flat_static reject an empty step-size table and slices that do not fit the arenas
    (a sum offset + count that wraps included) before anything touches the device."""
    import ctypes as C
    from paper_1910_05124_b200 import binding as B
    L = B.lib()
    fake = 4096                                                         # never dereferenced: every case fails first
    ar = B.pm_arenas(fake, fake, fake, fake, fake, None, 1 << 20)
    offs, cnts = (C.c_uint64 * 2)(0, 1024), (C.c_uint64 * 2)(1024, 1024)
    tf, tb = (C.c_int32 * 2)(3, 1), (C.c_int32 * 2)(0, 0)
    cfg, keep = B.make_config(n_stages=2, microbatch=1, compute="f32", optimizer="sgdm", alpha=0.01, alpha_by_step=[0.1, 0.2])
    cfg.alpha_len = 0
    st = L.pm_update_flat(C.byref(ar), offs, cnts, tf, tb, 2, C.byref(cfg), 0, C.c_void_p(fake), 1 << 20, None)
    assert L.pm_status_string(st) == b"PM_ERR_INVALID_ARG" and b"alpha_len" in L.pm_last_error(None)
    st = L.pm_update_flat_static(C.byref(ar), offs, cnts, tf, tb, 2, C.byref(cfg), 0, None)
    assert L.pm_status_string(st) == b"PM_ERR_INVALID_ARG" and b"alpha_len" in L.pm_update_flat_static_last_error()
    cfg.alpha_len = 2
    cnts[1] = (1 << 64) - 512                                            # offset + count wraps around
    st = L.pm_update_flat(C.byref(ar), offs, cnts, tf, tb, 2, C.byref(cfg), 0, C.c_void_p(fake), 1 << 20, None)
    assert L.pm_status_string(st) == b"PM_ERR_NOMEM"
