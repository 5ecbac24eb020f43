"""Workload descriptions and the recipes for their seeded synthetic data.

A workload is plain data: the stage list (which Linear layers ride in which
pipeline stage), the per-stage delays, the optimiser's hyper-parameters and
the seeds.  The recipes below turn a workload and a step index into tensors.
The teacher network that labels the MLP workloads is evaluated here, in
float64, with its own few lines of numpy; it is part of the data, not of the
training method.
"""
from dataclasses import dataclass, field
from typing import List

import numpy as np
from scipy.special import erf as _erf

from . import rng

# stream ids (purpose of a random draw)
_S_INIT, _S_TEACHER, _S_INPUT, _S_CALIB = 1, 2, 3, 500000
_CALIB_ROWS = 256
_CALIB_RMS = 1.0      # root-mean-square every pre-activation is calibrated to at initialisation
_S_UPD_W, _S_UPD_G, _S_UPD_M, _S_UPD_S, _S_UPD_D = 10, 11, 12, 13, 14


@dataclass
class LinearSpec:
    n_in: int
    n_out: int
    act: str  # 'relu' | 'gelu' | 'none'


@dataclass
class StageSpec:
    """One Transformer stage: pre-op, one Linear, post-op (see the encoder workload below)."""
    pre: str        # 'embed' | 'embed_dec' | 'ln' | 'none'
    n_in: int
    n_out: int
    act: str        # 'relu' | 'gelu' | 'none'
    post: str       # 'attention' | 'cross_attention' | 'skip_out' | 'residual' | 'none'
    src: str = "main"           # the Linear reads the main stream, or 'memory' (the encoder output)
    causal: bool = False        # 'attention': keys after the query are masked
    skip_hop: int = 1           # the skip tensor this stage emits goes to the stage skip_hop positions on
    emit_memory: bool = False   # the stage's output is also the memory of the cross-attention stages


@dataclass
class Workload:
    name: str
    stages: List[List[LinearSpec]]
    tau_fwd: List[int]
    tau_bkwd: List[int]
    microbatch: int
    compute: str = "f32"        # 'f32' | 'bf16' (GEMM operand type; state is always fp32)
    optimizer: str = "sgdm"     # 'sgdm' | 'adam'
    alpha: float = 0.01
    beta1: float = 0.9
    beta2: float = 0.98
    eps: float = 1e-8
    t1: bool = True
    K: int = 32
    t2: bool = True
    D: float = 0.5
    steps: int = 64
    seed: int = 191005124
    notes: str = field(default="")
    kind: str = "mlp"           # 'mlp' | 'encoder'
    stage_specs: List[StageSpec] = field(default_factory=list)   # encoder workloads
    n_heads: int = 0
    seq_len: int = 0
    vocab: int = 0
    d_model: int = 0

    @property
    def n_stages(self):
        return len(self.stage_specs) if self.kind == "encoder" else len(self.stages)


def pipemare_delays(P, n_micro=1):
    """Forward delays ceil((2(P-i)+1)/N) for i=1..P and zero backward delays (PipeMare row of Table 1)."""
    fwd = [-(-(2 * (P - i) + 1) // n_micro) for i in range(1, P + 1)]
    return fwd, [0] * P


def mlp_workload(name, P, width, linears_per_stage, act, microbatch, **kw):
    stages = [[LinearSpec(width, width, act) for _ in range(linears_per_stage)] for _ in range(P)]
    fwd, bkwd = pipemare_delays(P)
    return Workload(name=name, stages=stages, tau_fwd=fwd, tau_bkwd=bkwd, microbatch=microbatch, **kw)


def cfg1():
    """4-stage MLP, one Linear(256,256)+ReLU per stage, fp32, microbatch 32, 64 steps."""
    return mlp_workload("cfg1_mlp4_f32", 4, 256, 1, "relu", 32, compute="f32", optimizer="sgdm",
                        alpha=0.01, beta1=0.9, K=32, D=0.5, steps=64, seed=191005124 + 1)


def cfg3():
    """32-stage MLP, two Linear(1024,1024)+GELU per stage, bf16 GEMMs, microbatch 128, 500 steps."""
    return mlp_workload("cfg3_mlp32_bf16", 32, 1024, 2, "gelu", 128, compute="bf16", optimizer="sgdm",
                        alpha=0.01, beta1=0.9, K=125, D=0.5, steps=500, seed=191005124 + 3)


def cfg3_small(P=6, width=192, microbatch=40, steps=40, optimizer="sgdm"):
    """Same structure as cfg3 at a size the oracle runs in seconds (several tiles, ragged tails)."""
    return mlp_workload("cfg3_small", P, width, 2, "gelu", microbatch, compute="bf16", optimizer=optimizer,
                        alpha=0.01 if optimizer == "sgdm" else 5e-4, beta1=0.9, K=max(steps // 4, 1), D=0.5,
                        steps=steps, seed=191005124 + 33)


def round_to_bf16(x):
    """Round float values to the nearest bfloat16 (ties to even); returns float32 holding those values."""
    a = np.ascontiguousarray(x, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def _act(z, kind):
    if kind == "relu":
        return np.maximum(z, 0.0)
    if kind == "gelu":
        return 0.5 * z * (1.0 + _erf(z / np.sqrt(2.0)))
    return z


def _all_params(wl, stream):
    """Draw every Linear as N(0, 1/fan_in), then rescale layer by layer so that each
    pre-activation has unit root-mean-square on a fixed seeded calibration batch.

    A plain 64-layer GELU stack has no stable signal scale under a fixed-variance
    init (it vanishes or explodes with depth); calibrating on data keeps every
    layer's activations O(1) so that no part of the workload is degenerate.
    Biases start at zero.
    """
    n_in = wl.stages[0][0].n_in
    h = rng.normal(wl.seed, _S_CALIB + stream, _CALIB_ROWS * n_in).reshape(_CALIB_ROWS, n_in)
    out, index = [], 0
    for stage in wl.stages:
        tensors = []
        for spec in stage:
            w = rng.normal(wl.seed, stream + 1000 * (index + 1), spec.n_in * spec.n_out)
            w = w.reshape(spec.n_out, spec.n_in) / np.sqrt(spec.n_in)
            z = h @ w.T
            scale = _CALIB_RMS / np.sqrt(np.mean(z * z))
            w32 = (w * scale).astype(np.float32)
            h = _act(h @ w32.astype(np.float64).T, spec.act)
            tensors.append((w32, np.zeros(spec.n_out, dtype=np.float32)))
            index += 1
        out.append(tensors)
    return out


def init_stage_params(wl):
    """Initial student weights: per stage a list of (W[out,in], b[out]) float32 pairs."""
    return _all_params(wl, _S_INIT)


def teacher_params(wl):
    """Frozen teacher of the same architecture, drawn from a different stream."""
    return _all_params(wl, _S_TEACHER)


def batch(wl, t, teacher=None):
    """Microbatch t: x ~ N(0,1) of shape [M, in] and its teacher output y*, both float32.

    For bf16 workloads x is rounded to bfloat16-representable values first so
    that every consumer starts from identical operand bits.
    """
    n_in = wl.stages[0][0].n_in
    x = rng.normal(wl.seed, _S_INPUT + 16 * t, wl.microbatch * n_in).reshape(wl.microbatch, n_in)
    x = x.astype(np.float32)
    if wl.compute == "bf16":
        x = round_to_bf16(x)
    if teacher is None:
        teacher = teacher_params(wl)
    h = x.astype(np.float64)
    for stage, tensors in zip(wl.stages, teacher):
        for spec, (w, b) in zip(stage, tensors):
            h = _act(h @ w.astype(np.float64).T + b.astype(np.float64), spec.act)
    return x, h.astype(np.float32)


def update_sweep_case(n_params, P, optimizer="sgdm", seed=191005124 + 2, align=64):
    """Update-only workload: n_params split evenly over P stages, each slice padded to `align` elements.

    Returns a dict with per-stage (offset, count) in the padded flat arena, the
    delays, and float32 arrays w ~ N(0,1), g ~ N(0, sigma=1e-3), and small
    non-zero optimiser state so that no lane works on zeros or denormals.
    """
    base, rem = divmod(n_params, P)
    counts = [base + (1 if i < rem else 0) for i in range(P)]
    offsets, cur = [], 0
    for c in counts:
        offsets.append(cur)
        cur += -(-c // align) * align
    total = cur
    fwd, bkwd = pipemare_delays(P)

    def fill(stream, scale, positive=False):
        a = np.zeros(total, dtype=np.float32)
        for i, (o, c) in enumerate(zip(offsets, counts)):
            v = rng.normal(seed, stream + 100 * i, c) * scale
            a[o:o + c] = (v * v if positive else v).astype(np.float32)
        return a

    case = dict(n_params=n_params, P=P, optimizer=optimizer, offsets=offsets, counts=counts, total=total,
                tau_fwd=fwd, tau_bkwd=bkwd,
                w=fill(_S_UPD_W, 1.0), g=fill(_S_UPD_G, 1e-3), m=fill(_S_UPD_M, 1e-3),
                delta=fill(_S_UPD_D, 1e-4))
    if optimizer == "adam":
        case["s"] = fill(_S_UPD_S, 1e-3, positive=True)
    return case


# ---- Transformer encoder workloads -------------------------------------------------------------------------

_S_TOKENS, _S_ENC_INIT = 40, 50


def encoder_workload(name, n_layers, d_model, n_heads, d_ff, seq_len, batch, vocab, **kw):
    """Post-LN encoder, one stage per weight matrix: per layer [W_qkv + attention] [W_o + residual]
    [LN, W_1 + ReLU] [W_2 + residual]; the embedding rides with stage 1, each LayerNorm with the stage
    that follows it, and the vocabulary projection (with the final LayerNorm) is the last stage."""
    specs = []
    for layer in range(n_layers):
        specs.append(StageSpec("embed" if layer == 0 else "ln", d_model, 3 * d_model, "none", "attention"))
        specs.append(StageSpec("none", d_model, d_model, "none", "residual"))
        specs.append(StageSpec("ln", d_model, d_ff, "relu", "skip_out"))
        specs.append(StageSpec("none", d_ff, d_model, "none", "residual"))
    specs.append(StageSpec("ln", d_model, vocab, "none", "none"))
    P = len(specs)
    fwd, bkwd = pipemare_delays(P)
    return Workload(name=name, stages=[], tau_fwd=fwd, tau_bkwd=bkwd, microbatch=batch * seq_len, kind="encoder",
                    stage_specs=specs, n_heads=n_heads, seq_len=seq_len, vocab=vocab, d_model=d_model, **kw)


def cfg4():
    """Encoder, 6 layers, d_model 512, 8 heads, FFN 2048, sequence 128, microbatch 32 sequences, vocabulary 8192,
    bf16 GEMMs; target = input sequence reversed; Adam(0.9, 0.98), alpha 5e-4, K = 100, D = 0.1; 300 steps."""
    return encoder_workload("cfg4_encoder6_bf16", 6, 512, 8, 2048, 128, 32, 8192, compute="bf16", optimizer="adam",
                            alpha=5e-4, beta1=0.9, beta2=0.98, eps=1e-8, K=100, D=0.1, steps=300, seed=191005124 + 4)


def cfg4_small(compute="bf16", n_layers=2, d_model=64, n_heads=2, d_ff=128, seq_len=16, batch=3, vocab=96, steps=24):
    """Same structure as cfg4 at a size the oracle runs in seconds."""
    return encoder_workload("cfg4_small", n_layers, d_model, n_heads, d_ff, seq_len, batch, vocab, compute=compute,
                            optimizer="adam", alpha=5e-4, beta1=0.9, beta2=0.98, eps=1e-8, K=max(steps // 3, 1), D=0.1,
                            steps=steps, seed=191005124 + 44)


def encdec_workload(name, n_enc, n_dec, d_model, n_heads, d_ff, seq_len, batch, vocab, **kw):
    """Post-LN encoder-decoder, one stage per weight matrix.  Encoder layers as in encoder_workload; the last
    encoder stage also publishes the memory.  A decoder layer is seven stages: [W_qkv + causal attention]
    [W_o + residual] [LN, W_q, skip over two stages] [LN(memory), W_kv + cross-attention] [W_o + residual]
    [LN, W_1 + ReLU] [W_2 + residual]; the decoder's first stage embeds the decoder input (the target shifted
    right behind a begin-of-sequence id 0); the vocabulary projection with the final LayerNorm is the last stage.
    Source and target sequences have the same length."""
    specs = []
    for layer in range(n_enc):
        specs.append(StageSpec("embed" if layer == 0 else "ln", d_model, 3 * d_model, "none", "attention"))
        specs.append(StageSpec("none", d_model, d_model, "none", "residual"))
        specs.append(StageSpec("ln", d_model, d_ff, "relu", "skip_out"))
        specs.append(StageSpec("none", d_ff, d_model, "none", "residual", emit_memory=(layer == n_enc - 1)))
    for layer in range(n_dec):
        specs.append(StageSpec("embed_dec" if layer == 0 else "ln", d_model, 3 * d_model, "none", "attention", causal=True))
        specs.append(StageSpec("none", d_model, d_model, "none", "residual"))
        specs.append(StageSpec("ln", d_model, d_model, "none", "skip_out", skip_hop=2))
        specs.append(StageSpec("ln", d_model, 2 * d_model, "none", "cross_attention", src="memory"))
        specs.append(StageSpec("none", d_model, d_model, "none", "residual"))
        specs.append(StageSpec("ln", d_model, d_ff, "relu", "skip_out"))
        specs.append(StageSpec("none", d_ff, d_model, "none", "residual"))
    specs.append(StageSpec("ln", d_model, vocab, "none", "none"))
    P = len(specs)
    fwd, bkwd = pipemare_delays(P)
    return Workload(name=name, stages=[], tau_fwd=fwd, tau_bkwd=bkwd, microbatch=batch * seq_len, kind="encoder",
                    stage_specs=specs, n_heads=n_heads, seq_len=seq_len, vocab=vocab, d_model=d_model, **kw)


def cfg5():
    """Encoder-decoder, 12 + 12 layers, d_model 1024, 16 heads, FFN 4096, sequence 256, microbatch 16 sequences,
    vocabulary 32000, bf16 GEMMs; source ids Zipf(1.1), target = a fixed seeded permutation of the source ids;
    Adam(0.9, 0.98), alpha 7e-4, K = 1000, D = 0.1; 48 + 84 + 1 = 133 stages."""
    return encdec_workload("cfg5_encdec12_bf16", 12, 12, 1024, 16, 4096, 256, 16, 32000, compute="bf16", optimizer="adam",
                           alpha=7e-4, beta1=0.9, beta2=0.98, eps=1e-8, K=1000, D=0.1, steps=1200, seed=191005124 + 5)


def cfg5_cut(n_enc=7, n_dec=7, seq_len=256, batch=16, vocab=32000):
    """cfg5's widths and sequence shape (d_model 1024, 16 heads, FFN 4096, vocabulary 32000, 16 sequences of 256
    tokens per microbatch) with fewer layers: 7 + 7 layers (78 stages) is the deepest form whose activation rings
    fit one GPU's memory (150 GB of rings, 166 GB in all; 8 + 8 layers need 212 GB, the full 12 + 12 layers
    more than 450 GB)."""
    full = cfg5()
    return encdec_workload(f"cfg5_cut_{n_enc}+{n_dec}_bf16", n_enc, n_dec, 1024, 16, 4096, seq_len, batch, vocab, compute="bf16",
                           optimizer="adam", alpha=full.alpha, beta1=0.9, beta2=0.98, eps=1e-8, K=full.K, D=full.D,
                           steps=full.steps, seed=full.seed)


def cfg5_small(compute="bf16", n_enc=1, n_dec=1, d_model=64, n_heads=2, d_ff=128, seq_len=16, batch=3, vocab=96, steps=24):
    """Same structure as cfg5 at a size the oracle runs in seconds."""
    return encdec_workload("cfg5_small", n_enc, n_dec, d_model, n_heads, d_ff, seq_len, batch, vocab, compute=compute,
                           optimizer="adam", alpha=7e-4, beta1=0.9, beta2=0.98, eps=1e-8, K=max(steps // 3, 1), D=0.1,
                           steps=steps, seed=191005124 + 55)


def seq2seq_batch(wl, t):
    """Microbatch t of an encoder-decoder workload: (source ids, decoder input ids, target ids), each [batch*seq_len].
    Source ids are Zipf(1.1)-distributed ranks; the target is pi(source) for a permutation pi of the vocabulary fixed
    by the workload's seed; the decoder input is the target shifted right by one position behind id 0."""
    n_seq = wl.microbatch // wl.seq_len
    src = rng.zipf_ranks(wl.seed, _S_TOKENS + 16 * t, wl.microbatch, wl.vocab, 1.1).reshape(n_seq, wl.seq_len)
    order = np.argsort(rng.uniform01(wl.seed, _S_TOKENS + 5, wl.vocab), kind="stable")   # the permutation pi
    tgt = order[src]
    dec_in = np.concatenate([np.zeros((n_seq, 1), dtype=np.int64), tgt[:, :-1]], axis=1)
    return src.reshape(-1).astype(np.int64), dec_in.reshape(-1).astype(np.int64), tgt.reshape(-1).astype(np.int64)


def init_encoder_params(wl):
    """Per stage the tensors [table] [gain, bias] W b (float32): W ~ N(0, 1/fan_in), table ~ N(0, 1/d_model),
    biases 0, LayerNorm gain 1 and bias 0."""
    out = []
    for i, sp in enumerate(wl.stage_specs):
        tensors = []
        if sp.pre in ("embed", "embed_dec"):
            e = rng.normal(wl.seed, _S_ENC_INIT + (7 if sp.pre == "embed" else 8), wl.vocab * wl.d_model) / np.sqrt(wl.d_model)
            tensors.append(e.reshape(wl.vocab, wl.d_model).astype(np.float32))
        if sp.pre == "ln":
            tensors += [np.ones(sp.n_in, dtype=np.float32), np.zeros(sp.n_in, dtype=np.float32)]
        w = rng.normal(wl.seed, _S_ENC_INIT + 1000 * (i + 1), sp.n_in * sp.n_out) / np.sqrt(sp.n_in)
        tensors += [w.reshape(sp.n_out, sp.n_in).astype(np.float32), np.zeros(sp.n_out, dtype=np.float32)]
        out.append(tensors)
    return out


def token_batch(wl, t):
    """Microbatch t: ids uniform on [0, vocab) of shape [batch*seq_len]; target = each sequence reversed."""
    n_seq = wl.microbatch // wl.seq_len
    ids = rng.randint(wl.seed, _S_TOKENS + 16 * t, wl.microbatch, wl.vocab).reshape(n_seq, wl.seq_len)
    return ids.reshape(-1).astype(np.int64), ids[:, ::-1].reshape(-1).astype(np.int64)


_S_DELAYS = 900000


def stochastic_delays(seed, n_steps, means, tau_max):
    """Integer gradient delays of the stage-wise stochastic delay model (Appendix E): for every step and stage a draw
    from the exponential distribution with the stage's mean, truncated below tau_max + 1 (inverse CDF on a counter-based
    uniform) and rounded down.  Returns a list of n_steps lists of len(means) integers in [0, tau_max]."""
    P = len(means)
    u = rng.uniform01(seed, _S_DELAYS, n_steps * P).reshape(n_steps, P)
    mu = np.maximum(np.asarray(means, dtype=np.float64), 1e-9)[None, :]
    x = -mu * np.log(1.0 - u * (1.0 - np.exp(-float(tau_max + 1) / mu)))
    return np.minimum(np.floor(x).astype(np.int64), tau_max).tolist()
