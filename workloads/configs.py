"""The five benchmark configurations and the small scenario cases, as metadata.

cfg1..cfg5 restate the shapes and parallelism changes the benchmark definition names; the
scenario cases restate the parallelism transitions the paper itself exercises (Sec. 6.4 /
Appendix E: PP, TP, DP and hybrid changes from TP1.DP4.PP4; Fig. 2: 8 -> 6 -> 4 workers;
Table 3: ZeRO-2 32 -> 64 and 128 -> 64 ranks, DP75 <-> DP150) on a tiny model.
"""
from __future__ import annotations

from typing import Callable, Dict, List

from .layouts import (ModelSpec, Parallelism, ReshardCase, StateKinds, build_state, gpt_model, llama_model,
                      moe_model, reshard_case)
from .meta import DTYPE_BF16, DTYPE_F32

MIXED = StateKinds()  # bf16 params + fp32 master / exp_avg / exp_avg_sq
PARAMS_ONLY = StateKinds(optim=())
OPTIM_ONLY = StateKinds(param_dtype=None)
MOE_KINDS = StateKinds(optim=("exp_avg",))
F32_PARAMS = StateKinds(param_dtype=(4, DTYPE_F32), optim=())  # parameters kept in binary32 (master copy)


def cfg1(fill: str = "uniform") -> ReshardCase:
    m = gpt_model("gpt-tiny", L=2, H=256, F=1024, V=1024, P=128)
    return reshard_case("cfg1-tiny-gpt", m, Parallelism(tp=2, dp=2, zero="zero1"),
                        Parallelism(tp=1, dp=4, zero="zero1"), MIXED, fill, seed=0)


def cfg2(layers: int = 24) -> ReshardCase:
    """GPT-3 1.3B shape.  `layers` < 24 keeps the per-layer shapes and shrinks the depth (used
    for profiler captures that must stay small)."""
    m = gpt_model("gpt3-1.3b", L=layers, H=2048, F=8192, V=50304, P=2048)
    return reshard_case("cfg2-gpt3-1.3b" + ("" if layers == 24 else f"-L{layers}"), m,
                        Parallelism(tp=4, pp=2, dp=2, zero="zero1"),
                        Parallelism(tp=2, pp=1, dp=4, zero="zero1"), MIXED, "normal", seed=20145)


def cfg3(layers: int = 32) -> ReshardCase:
    m = llama_model("llama3-8b", L=layers, H=4096, nq=32, nkv=8, F=14336, V=128256, fused=True, tied=False)
    return reshard_case("cfg3-llama3-8b" + ("" if layers == 32 else f"-L{layers}"), m,
                        Parallelism(tp=8), Parallelism(tp=2), PARAMS_ONLY, "normal", seed=20146)


def cfg4(layers: int = 28) -> ReshardCase:
    m = llama_model("llama-3b-fsdp", L=layers, H=3072, nq=24, nkv=8, F=8192, V=128256, fused=False,
                    tied=True, fsdp_units=True)
    return reshard_case("cfg4-llama-3b-fsdp" + ("" if layers == 28 else f"-L{layers}"), m,
                        Parallelism(dp=64, zero="fsdp"), Parallelism(dp=48, zero="fsdp"),
                        OPTIM_ONLY, "index", seed=20147)


def cfg5(layers: int = 16) -> ReshardCase:
    m = moe_model("moe-64e", L=layers, H=2048, E=64, F=1408, V=32768)
    return reshard_case("cfg5-moe" + ("" if layers == 16 else f"-L{layers}"), m,
                        Parallelism(ep=8), Parallelism(ep=4), MOE_KINDS, "uniform", seed=20148)


def cfg4_odd(layers: int = 28) -> ReshardCase:
    """Unscored stress variant of cfg4: DP61 -> DP47, so flat slices are 1,650,319 and 2,141,903
    elements long (both odd): source and target byte offsets differ by odd multiples of 4 bytes
    and no copy can use 16-byte accesses on both sides."""
    m = llama_model("llama-3b-fsdp", L=layers, H=3072, nq=24, nkv=8, F=8192, V=128256, fused=False,
                    tied=True, fsdp_units=True)
    return reshard_case("cfg4-odd-dp61-to-dp47" + ("" if layers == 28 else f"-L{layers}"), m,
                        Parallelism(dp=61, zero="fsdp"), Parallelism(dp=47, zero="fsdp"),
                        OPTIM_ONLY, "index", seed=20149)


def narrow_rows(layers: int = 4, cols: int = 256) -> ReshardCase:
    """Unscored stress: `layers` bf16 tensors of shape (2^28 / cols, cols) split along dim 1, two
    ways saved and four ways wanted, so every copy is a rectangle with rows of cols / 2 bytes
    (128 bytes by default) and 512 MB per tensor."""
    from .layouts import ModelSpec, TensorSpec

    m = ModelSpec("narrow", [TensorSpec(f"t{i}.weight", ((1 << 28) // cols, cols), "row", layer=i) for i in range(layers)], layers)
    return reshard_case(f"narrow-rows-{cols // 2}B-x{layers}", m, Parallelism(tp=2), Parallelism(tp=4), PARAMS_ONLY, "index",
                        seed=20150)


def odd_gpt(layers: int = 12) -> ReshardCase:
    """Unscored stress: a GPT with hidden 3000, FFN 12000 and the 50257-token vocabulary, bf16
    parameters, TP3 -> TP2: the splits are uneven and row-parallel weights are cut at odd element
    counts, so most two-dimensional pieces are only 2-, 4- or 8-byte aligned."""
    m = gpt_model("gpt-odd", L=layers, H=3000, F=12000, V=50257, P=1024)
    return reshard_case(f"odd-gpt-tp3-to-tp2-L{layers}", m, Parallelism(tp=3), Parallelism(tp=2), PARAMS_ONLY, "index",
                        seed=20151)


STRESS: Dict[str, Callable[..., ReshardCase]] = {"cfg4odd": cfg4_odd, "narrow": narrow_rows, "oddgpt": odd_gpt,
                                                   "evalmerge": lambda layers=32: eval_merge(layers)}  # defined below

CONFIGS: Dict[str, Callable[..., ReshardCase]] = {
    "cfg1": cfg1, "cfg2": cfg2, "cfg3": cfg3, "cfg4": cfg4, "cfg5": cfg5}

# closed-form byte totals of the full-size configurations (sum over entries)
EXPECTED_TOTALS = {
    "cfg1": (26_249_216, 37_498_880),
    "cfg2": (18_421_473_280, 26_406_256_640),
    "cfg3": (16_060_522_496, 16_061_054_976),
    "cfg4": (38_552_997_888, 38_552_997_888),
    "cfg5": (55_579_127_808, 62_865_850_368),
}


# --------------------------------------------------------------------------- small scenarios
def small_gpt() -> ModelSpec:
    return gpt_model("gpt-s", L=8, H=64, F=256, V=512, P=32)


def small_llama(fused: bool = True) -> ModelSpec:
    return llama_model("llama-s", L=4, H=128, nq=8, nkv=2, F=352, V=1000, fused=fused, tied=False)


def scenario_cases() -> List[ReshardCase]:
    g = small_gpt()
    base = Parallelism(tp=1, dp=4, pp=4, zero="zero1")
    out = [
        reshard_case("pp4-to-pp8", g, base, Parallelism(tp=1, dp=4, pp=8, zero="zero1"), MIXED),
        reshard_case("tp1-to-tp2", g, base, Parallelism(tp=2, dp=4, pp=4, zero="zero1"), MIXED),
        reshard_case("dp4-to-dp8", g, base, Parallelism(tp=1, dp=8, pp=4, zero="zero1"), MIXED),
        reshard_case("hybrid", g, base, Parallelism(tp=2, dp=8, pp=2, zero="zero1"), MIXED),
        reshard_case("workers-8-to-6", g, Parallelism(dp=8, zero="zero1"), Parallelism(dp=6, zero="zero1"), MIXED),
        reshard_case("workers-6-to-4", g, Parallelism(dp=6, zero="zero1"), Parallelism(dp=4, zero="zero1"), MIXED),
        reshard_case("dp75-to-dp150", g, Parallelism(tp=4, dp=75, zero="zero1"),
                     Parallelism(tp=4, dp=150, zero="zero1"), OPTIM_ONLY),
        reshard_case("dp150-to-dp75", g, Parallelism(tp=4, dp=150, zero="zero1"),
                     Parallelism(tp=4, dp=75, zero="zero1"), OPTIM_ONLY),
    ]
    l = small_llama()
    out += [
        reshard_case("llama-tp8-to-tp2", l, Parallelism(tp=8), Parallelism(tp=2), PARAMS_ONLY),
        reshard_case("llama-tp2-to-tp8", l, Parallelism(tp=2), Parallelism(tp=8), PARAMS_ONLY),
        reshard_case("fsdp-32-to-64", llama_model("llama-f", 3, 96, 6, 2, 200, 777, fused=False, tied=True,
                                                  fsdp_units=True),
                     Parallelism(dp=32, zero="fsdp"), Parallelism(dp=64, zero="fsdp"), OPTIM_ONLY),
        reshard_case("fsdp-128-to-64", llama_model("llama-f", 3, 96, 6, 2, 200, 777, fused=False, tied=True,
                                                   fsdp_units=True),
                     Parallelism(dp=128, zero="fsdp"), Parallelism(dp=64, zero="fsdp"), OPTIM_ONLY),
        reshard_case("moe-ep8-to-ep4", moe_model("moe-s", 2, 64, 16, 48, 256), Parallelism(ep=8),
                     Parallelism(ep=4), MOE_KINDS),
        # odd sizes: vocabulary 50257 and hidden 1000 split three ways (uneven), bf16 rows cut at odd
        # element counts, so two-dimensional pieces are only 2-byte aligned
        reshard_case("odd-gpt-tp3-to-tp2", gpt_model("gpt-odd", L=1, H=1000, F=4000, V=50257, P=77), Parallelism(tp=3),
                     Parallelism(tp=2), PARAMS_ONLY),
        stacked_experts_case(),
    ]
    return out


def stacked_experts_case() -> ReshardCase:
    """Experts stacked in one 3-D tensor [E, F, H]: saved split along dim 0 over 4 ranks, wanted
    as six flat slices of the whole stack (boundaries inside rows of the middle experts)."""
    from .meta import FLAT_SLICE, ShardMeta, ShardedState

    E, F, H, isz = 8, 24, 40, 4
    shape = (E, F, H)
    src = ShardedState([ShardMeta("experts.w", isz, DTYPE_F32, shape, (2 * r, 0, 0), (2, F, H), r, 256) for r in range(4)],
                       [256 + 2 * F * H * isz] * 4)
    n = E * F * H
    cut = -(-n // 6)
    dst = ShardedState([ShardMeta("experts.w", isz, DTYPE_F32, shape, (0, 0, 0), shape, r, 0, FLAT_SLICE, r * cut,
                                  min(n, (r + 1) * cut)) for r in range(6)],
                       [(min(n, (r + 1) * cut) - r * cut) * isz for r in range(6)])
    return ReshardCase("stacked-experts-3d", src, dst, "index", 3)


# --------------------------------------------------------------------------- element conversion
def convert_case(name: str, model: ModelSpec, src_par: Parallelism, dst_par: Parallelism, narrow: bool = True,
                 fill: str = "index", seed: int = 0, flat: bool = False) -> ReshardCase:
    """Parameters saved in binary32 and wanted in bfloat16 under another parallelism (narrow),
    or the reverse.  Not one of the paper's workloads: the paper moves bytes only."""
    if flat:  # one optimizer state per parameter, flat-partitioned (ZeRO / FSDP), in either type
        wide, slim = (StateKinds(param_dtype=None, optim=("master",), optim_dtype=d) for d in ((4, DTYPE_F32), (2, DTYPE_BF16)))
    else:
        wide, slim = F32_PARAMS, PARAMS_ONLY
    a, b = (wide, slim) if narrow else (slim, wide)
    tags = (1, DTYPE_F32, DTYPE_BF16) if narrow else (2, DTYPE_BF16, DTYPE_F32)
    return ReshardCase(name, build_state(model, src_par, a, dedup=True), build_state(model, dst_par, b, dedup=False),
                       fill, seed, convert=tags)


def convert_cases() -> List[ReshardCase]:
    g, l = small_gpt(), small_llama()
    odd = gpt_model("gpt-odd", L=2, H=60, F=150, V=251, P=17)  # odd sizes: rows start at every alignment
    f = llama_model("llama-f", 3, 96, 6, 2, 200, 777, fused=False, tied=True, fsdp_units=True)
    return [
        convert_case("narrow-gpt-tp1-to-tp2", g, Parallelism(tp=1, dp=2), Parallelism(tp=2, dp=2)),
        convert_case("narrow-llama-tp8-to-tp2", l, Parallelism(tp=8), Parallelism(tp=2)),
        convert_case("narrow-odd-tp3-to-tp2", odd, Parallelism(tp=3), Parallelism(tp=2)),
        convert_case("widen-llama-tp2-to-tp8", l, Parallelism(tp=2), Parallelism(tp=8), narrow=False),
        convert_case("widen-odd-tp2-to-tp3", odd, Parallelism(tp=2), Parallelism(tp=3), narrow=False),
        convert_case("narrow-fsdp-5-to-3", f, Parallelism(dp=5, zero="fsdp"), Parallelism(dp=3, zero="fsdp"), flat=True),
        convert_case("widen-zero1-dp3-to-dp4", g, Parallelism(tp=2, dp=3, zero="zero1"), Parallelism(tp=1, dp=4, zero="zero1"),
                     narrow=False, flat=True),
    ]


def eval_merge(layers: int = 32) -> ReshardCase:
    """Unscored: the Llama-3-8B shapes of cfg3 with binary32 parameters saved under TP8 and wanted in
    bfloat16 under TP2 (32 GB read, 16 GB written)."""
    m = llama_model("llama3-8b", L=layers, H=4096, nq=32, nkv=8, F=14336, V=128256, fused=True, tied=False)
    return convert_case("eval-merge-llama3-8b-f32-to-bf16" + ("" if layers == 32 else f"-L{layers}"), m,
                        Parallelism(tp=8), Parallelism(tp=2), True, "normal", 20150)
