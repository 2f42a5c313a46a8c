"""Workload shapes of the H-Spec block-parallel draft step.

Each config is a plain dict of integers/floats.  Symbols follow the paper's
notation (Sec. 3.3, App. B.1): D = hidden size, r = fusion rank, Di = Mamba
inner size, P = Mamba head dim, N = state dim, G = B/C groups, Hq/Hkv =
query/KV heads, dh = attention head dim, F = MLP width, V = vocabulary,
L = drafter layers, B = concurrent requests, k = block positions.
"""
import copy

_MODEL_8B = dict(
    D=4096, n_fuse=1, r=4096, L=2, has_attn=[1, 1], kv_slot=[0, 1], n_slots=2,
    Di=8192, P=64, N=128, G=4, d_conv=4, dt_rank=0,
    Hq=32, Hkv=8, dh=128, rope_theta=1.0e6, window=0, qk_norm=1,
    F=14336, V=128256, rms_eps=1e-6, page_size=16,
)
_MODEL_32B = dict(
    D=5120, n_fuse=1, r=5120, L=2, has_attn=[1, 1], kv_slot=[0, 1], n_slots=2,
    Di=10240, P=64, N=128, G=4, d_conv=4, dt_rank=0,
    Hq=64, Hkv=8, dh=128, rope_theta=1.0e6, window=0, qk_norm=1,
    F=25600, V=152064, rms_eps=1e-6, page_size=16,
)
_MODEL_TINY = dict(
    D=256, n_fuse=1, r=256, L=1, has_attn=[1], kv_slot=[0], n_slots=1,
    Di=512, P=64, N=16, G=1, d_conv=4, dt_rank=16,
    Hq=4, Hkv=2, dh=64, rope_theta=1.0e4, window=0, qk_norm=1,
    F=1024, V=1024, rms_eps=1e-6, page_size=16,
)
# The paper's own drafter shape for an 8B-class target (App. B.1): 48 Mamba
# heads of 64, state = groups = conv = 4, expansion 1, five fused hidden
# states, three attention layers + one Mamba-MLP layer, window 2048.
_MODEL_PAPER_8B = dict(
    D=4096, n_fuse=5, r=4096, L=4, has_attn=[1, 1, 1, 0], kv_slot=[0, 1, 2, -1],
    n_slots=3, Di=3072, P=64, N=4, G=4, d_conv=4, dt_rank=0,
    Hq=32, Hkv=8, dh=128, rope_theta=1.0e6, window=2048, qk_norm=1,
    F=12288, V=151936, rms_eps=1e-6, page_size=16, markov_rank=256,
)

CONFIGS = {
    "tiny": dict(_MODEL_TINY, name="tiny", B=1, k=8, ctx=("const", 256, 256)),
    "latency_8b": dict(_MODEL_8B, name="latency_8b", B=1, k=16, ctx=("const", 2048, 2048)),
    "serving_8b": dict(_MODEL_8B, name="serving_8b", B=32, k=16, ctx=("uniform", 512, 8192)),
    "conc128_32b": dict(_MODEL_32B, name="conc128_32b", B=128, k=16, ctx=("loguniform", 1024, 32768)),
    # the concurrency-128 workload with the drafter predicting over a pruned 32 000-token vocabulary (App. B.2)
    "conc128_32b_v32k": dict(_MODEL_32B, name="conc128_32b_v32k", V_draft=32000, B=128, k=16, ctx=("loguniform", 1024, 32768)),
    "paper_8b": dict(_MODEL_PAPER_8B, name="paper_8b", B=32, k=8, ctx=("uniform", 512, 8192)),
    # the concurrency-128 workload with the rank-256 causal-correction head behind the LM head (Sec. 3.3.3, App. B.1)
    "conc128_32b_markov": dict(_MODEL_32B, name="conc128_32b_markov", markov_rank=256, B=128, k=16,
                               ctx=("loguniform", 1024, 32768)),
}


def sweep_config(B, k):
    """One cell of the concurrency x block-size sweep on the 8B-class drafter."""
    return dict(_MODEL_8B, name=f"sweep_8b_B{B}_k{k}", B=B, k=k, ctx=("uniform", 1024, 16384))


def get_config(name, **overrides):
    """Config by name: one of CONFIGS, or a sweep cell 'sweep_8b_B<B>_k<k>'."""
    if name.startswith("sweep_8b_B"):
        B, k = name[len("sweep_8b_B"):].split("_k")
        cfg = sweep_config(int(B), int(k))
        cfg.update(overrides)
        return derived(cfg)
    cfg = copy.deepcopy(CONFIGS[name])
    cfg.update(overrides)
    return derived(cfg)


def derived(cfg):
    """Fill in the sizes that follow from the others (no arithmetic of the method)."""
    cfg = dict(cfg)
    assert cfg["Di"] % cfg["P"] == 0
    cfg["H"] = cfg["Di"] // cfg["P"]
    assert cfg["H"] % cfg["G"] == 0 and cfg["Hq"] % cfg["Hkv"] == 0
    cfg["d_S"] = cfg["H"] * cfg["P"] * cfg["N"]
    cfg["d_xBC"] = cfg["Di"] + 2 * cfg["G"] * cfg["N"]
    cfg["d_dt"] = cfg["dt_rank"] if cfg["dt_rank"] > 0 else cfg["H"]
    cfg["d_in_proj"] = cfg["Di"] + cfg["d_xBC"] + cfg["d_dt"]
    cfg["d_qkv"] = (cfg["Hq"] + 2 * cfg["Hkv"]) * cfg["dh"]
    cfg.setdefault("mask_id", cfg["V"] - 1)
    cfg.setdefault("markov_rank", 0)
    return cfg
