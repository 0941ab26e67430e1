"""Synthetic workload recipes: tensor lists, optimizer groups and run settings.

These are shapes and settings only (what a training job would hand to the
optimizer), shared by the tests and the benchmark so that the CUDA library and
the CPU oracle are driven with the same seeded inputs.  No spread, schedule,
optimizer or controller arithmetic lives here.

The paper's backbone is not described (its data and model are proprietary), so
the "large model" workloads use the parameter list of a GPT-2-style decoder with
a tied output head, and the four optimizer groups the paper names
(embedding, no_decay, non_embedding, transformer).  Group membership is this
repository's choice: embeddings; all biases and LayerNorm tensors (no weight
decay); MLP matrices; attention matrices.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence, Tuple

GROUP_EMBEDDING = 0
GROUP_NO_DECAY = 1
GROUP_NON_EMBEDDING = 2
GROUP_TRANSFORMER = 3
GROUP_NAMES = ("embedding", "no_decay", "non_embedding", "transformer")

OPT_SGD = 0
OPT_ADAMW = 1
DTYPE_F32 = 0
DTYPE_BF16 = 1
SCHED_CONSTANT = 0
SCHED_ONECYCLE_COS = 1
SCHED_ONECYCLE_LINEAR = 2


@dataclass(frozen=True)
class TensorSpec:
    name: str
    numel: int
    group: int


@dataclass(frozen=True)
class Workload:
    name: str
    n_replicas: int
    tensors: Tuple[TensorSpec, ...]
    n_groups: int
    optimizer: int
    grad_dtype: int
    # optimizer constants
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    momentum: float = 0.0   # SGD momentum (0 = plain Eq. 2)
    weight_decay: Tuple[float, ...] = (0.0,)
    # base schedule
    sched_kind: int = SCHED_CONSTANT
    max_lr: Tuple[float, ...] = (1e-2,)
    total_steps: int = 16
    pct_start: float = 0.3
    div_factor: float = 25.0
    final_div_factor: float = 1e4
    # HDET
    alpha_lr: float = 0.0
    alpha_wd: float = 0.0
    sync_interval: int = 1
    reshuffle: int = 1
    # auto-LR controller
    autolr: int = 0
    warmup_steps: int = 0
    ctrl_beta: float = 0.9
    ctrl_sigma: float = 0.1
    ctrl_lambda: float = 0.5
    f_div: float = 25.0
    f_final: float = 1.0
    auto_wd: int = 0        # controller also on the weight-decay channel (Remark 1)
    # inputs
    seed: int = 1
    param_sigma: float = 0.02
    grad_sigma: float = 1e-3
    loss_kind: str = "uniform"  # "uniform": U(2,3); "rank": 3.0 - 0.1*offset + N(0, 0.01^2)
    align_elems: int = 8  # arena offsets of tensors are multiples of this many elements

    @property
    def numel(self) -> int:
        return sum(t.numel for t in self.tensors)

    def arena_offsets(self) -> List[int]:
        """Element offset of every tensor inside one replica's arena."""
        offs, cur = [], 0
        a = self.align_elems
        for t in self.tensors:
            offs.append(cur)
            cur += (t.numel + a - 1) // a * a
        return offs

    def arena_numel(self) -> int:
        """Elements per replica in the arena (padding included)."""
        a = self.align_elems
        return sum((t.numel + a - 1) // a * a for t in self.tensors)


def decoder_tensor_list(n_layers: int, d: int, ffn: int, vocab: int, ctx: int) -> Tuple[TensorSpec, ...]:
    """Parameter list of a GPT-2-style decoder with a tied output head (12*L + 4 tensors)."""
    ts: List[TensorSpec] = [
        TensorSpec("wte", vocab * d, GROUP_EMBEDDING),
        TensorSpec("wpe", ctx * d, GROUP_EMBEDDING),
    ]
    for l in range(n_layers):
        p = f"h{l}."
        ts += [
            TensorSpec(p + "ln1.w", d, GROUP_NO_DECAY),
            TensorSpec(p + "ln1.b", d, GROUP_NO_DECAY),
            TensorSpec(p + "qkv.w", d * 3 * d, GROUP_TRANSFORMER),
            TensorSpec(p + "qkv.b", 3 * d, GROUP_NO_DECAY),
            TensorSpec(p + "proj.w", d * d, GROUP_TRANSFORMER),
            TensorSpec(p + "proj.b", d, GROUP_NO_DECAY),
            TensorSpec(p + "ln2.w", d, GROUP_NO_DECAY),
            TensorSpec(p + "ln2.b", d, GROUP_NO_DECAY),
            TensorSpec(p + "fc.w", d * ffn, GROUP_NON_EMBEDDING),
            TensorSpec(p + "fc.b", ffn, GROUP_NO_DECAY),
            TensorSpec(p + "fc2.w", ffn * d, GROUP_NON_EMBEDDING),
            TensorSpec(p + "fc2.b", d, GROUP_NO_DECAY),
        ]
    ts += [TensorSpec("lnf.w", d, GROUP_NO_DECAY), TensorSpec("lnf.b", d, GROUP_NO_DECAY)]
    return tuple(ts)


def _wd4(wd: float) -> Tuple[float, ...]:
    out = [wd] * 4
    out[GROUP_NO_DECAY] = 0.0
    return tuple(out)


def config1() -> Workload:
    """N=4, one flat fp32 tensor of 1e6 elements, plain SGD, constant LR, T=4, 16 steps."""
    return Workload(
        name="config1_sgd_flat_1M",
        n_replicas=4,
        tensors=(TensorSpec("flat", 1_000_000, 0),),
        n_groups=1,
        optimizer=OPT_SGD,
        grad_dtype=DTYPE_F32,
        weight_decay=(0.0,),
        sched_kind=SCHED_CONSTANT,
        max_lr=(1e-2,),
        total_steps=16,
        alpha_lr=0.2,
        sync_interval=4,
        autolr=0,
        seed=1,
        grad_sigma=1e-2,
        loss_kind="uniform",
    )


def config2() -> Workload:
    """N=8, 12 x ([1024,2048], [2048]) = 25,190,400 params, AdamW, OneCycle 1000 steps, T=50, auto-LR."""
    ts = []
    for k in range(12):
        ts.append(TensorSpec(f"w{k}", 1024 * 2048, 0))
        ts.append(TensorSpec(f"b{k}", 2048, 0))
    return Workload(
        name="config2_adamw_25M",
        n_replicas=8,
        tensors=tuple(ts),
        n_groups=1,
        optimizer=OPT_ADAMW,
        grad_dtype=DTYPE_BF16,
        weight_decay=(0.01,),
        sched_kind=SCHED_ONECYCLE_COS,
        max_lr=(3e-4,),
        total_steps=1000,
        alpha_lr=0.3,
        sync_interval=50,
        autolr=1,
        warmup_steps=300,
        seed=2,
        loss_kind="rank",
    )


def _decoder_workload(name, n, layers, d, ffn, ctx, steps, alpha, T, autolr, seed, wd=0.01, alpha_wd=0.0):
    return Workload(
        name=name,
        n_replicas=n,
        tensors=decoder_tensor_list(layers, d, ffn, 50257, ctx),
        n_groups=4,
        optimizer=OPT_ADAMW,
        grad_dtype=DTYPE_BF16,
        weight_decay=_wd4(wd),
        sched_kind=SCHED_ONECYCLE_COS,
        max_lr=(3e-4,) * 4,
        total_steps=steps,
        alpha_lr=alpha,
        alpha_wd=alpha_wd,
        sync_interval=T,
        autolr=autolr,
        warmup_steps=int(round(0.3 * steps)) if autolr else 0,
        seed=seed,
        loss_kind="rank",
    )


def config3() -> Workload:
    """N=8, 24-layer decoder d=1024 (354,823,168 params, 292 tensors), T=100, 500 steps, auto-LR."""
    return _decoder_workload("config3_decoder_350M", 8, 24, 1024, 4096, 1024, 500, 0.3, 100, 1, 3)


def config4() -> Workload:
    """N=8, 24-layer decoder d=2048 (1,315,723,264 params), T=1 (converge every step), 50 steps."""
    return _decoder_workload("config4_decoder_1p3B", 8, 24, 2048, 8192, 2048, 50, 0.5, 1, 0, 4)


def config5(sync_interval: int = 10) -> Workload:
    """N=16, 12-layer decoder d=768 (124,439,808 params), LR spread 0.3 and wd 0.05 +-50 %, 300 steps."""
    w = _decoder_workload(
        f"config5_decoder_125M_T{sync_interval}", 16, 12, 768, 3072, 1024, 300, 0.3, sync_interval, 1, 5,
        wd=0.05, alpha_wd=0.5,
    )
    return w


def scaled_decoder(base: Workload, layers: int, d: int, ffn: int, vocab: int, ctx: int, steps: Optional[int] = None,
                   name: Optional[str] = None) -> Workload:
    """A smaller decoder with the settings of ``base`` (for tests that must finish in seconds)."""
    s = base.total_steps if steps is None else steps
    return replace(
        base,
        name=name or (base.name + "_scaled"),
        tensors=decoder_tensor_list(layers, d, ffn, vocab, ctx),
        total_steps=s,
        warmup_steps=int(round(0.3 * s)) if base.autolr else 0,
    )


def ragged_workload(n_replicas: int = 3, optimizer: int = OPT_ADAMW, grad_dtype: int = DTYPE_BF16,
                    align_elems: int = 8, numels: Sequence[int] = (1, 7, 8, 33, 1023, 1024, 2049, 4097, 12289, 5),
                    n_groups: int = 2) -> Workload:
    """Odd-sized tensors: tails shorter than a vector, exact tile multiples, one element."""
    ts = tuple(TensorSpec(f"t{k}", int(n), k % n_groups) for k, n in enumerate(numels))
    return Workload(
        name=f"ragged_N{n_replicas}_a{align_elems}",
        n_replicas=n_replicas,
        tensors=ts,
        n_groups=n_groups,
        optimizer=optimizer,
        grad_dtype=grad_dtype,
        weight_decay=tuple(0.01 * (g + 1) for g in range(n_groups)),
        sched_kind=SCHED_ONECYCLE_COS,
        max_lr=tuple(3e-4 * (g + 1) for g in range(n_groups)),
        total_steps=12,
        alpha_lr=0.25,
        alpha_wd=0.4,
        sync_interval=3,
        autolr=1,
        warmup_steps=4,
        seed=11,
        grad_sigma=1e-3,
        loss_kind="rank",
        align_elems=align_elems,
    )


ALL_CONFIGS = {
    "config1": config1,
    "config2": config2,
    "config3": config3,
    "config4": config4,
    "config5": config5,
}
