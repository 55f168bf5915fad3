"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module draws random tensors of the shapes and value distributions of the
benchmark configurations and nothing else: it holds none of the method's
arithmetic (no quantiser, no Philox, no perturbation, no model maths) and
imports neither the CUDA binding nor the CPU oracle.  All tensors are CPU torch
tensors; 16-bit values are torch.bfloat16.
"""
import torch

CONFIGS = {
    # Tiny decoder-only LM (2 layers, d 256, 4 heads, gated FFN 688, vocab 1024).
    "tiny": dict(arch="llama", n_layers=2, d_model=256, n_heads=4, d_ffn=688, vocab=1024,
                 max_seq=64, norm_eps=1e-5, rope_theta=10000.0, batch=4, seq=64,
                 eps=1e-3, lr=1e-5, clip=100.0),
    # Tiny OPT-style variant (LayerNorm, learned positions, ReLU, biases) for parity tests.
    "tiny_opt": dict(arch="opt", n_layers=2, d_model=256, n_heads=4, d_ffn=1024, vocab=1000,
                     max_seq=64, norm_eps=1e-5, rope_theta=0.0, batch=4, seq=48,
                     eps=1e-3, lr=1e-5, clip=10.0),
    # Tiny variant with head dimension 128 and several ragged attention blocks (parity tests).
    "tiny_dh128": dict(arch="llama", n_layers=2, d_model=256, n_heads=2, d_ffn=688, vocab=1024,
                       max_seq=200, norm_eps=1e-5, rope_theta=10000.0, batch=2, seq=200,
                       eps=1e-3, lr=1e-5, clip=100.0),
    "llama7b": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008,
                    vocab=32000, max_seq=256, norm_eps=1e-5, rope_theta=10000.0,
                    batch=16, seq=256, eps=1e-3, lr=1e-5, clip=100.0),
    "llama13b": dict(arch="llama", n_layers=40, d_model=5120, n_heads=40, d_ffn=13824,
                     vocab=32000, max_seq=512, norm_eps=1e-5, rope_theta=10000.0,
                     batch=8, seq=512, eps=1e-3, lr=1e-5, clip=100.0),
    "opt6.7b": dict(arch="opt", n_layers=32, d_model=4096, n_heads=32, d_ffn=16384,
                    vocab=50272, max_seq=128, norm_eps=1e-5, rope_theta=0.0,
                    batch=32, seq=128, eps=1e-3, lr=1e-5, clip=10.0),
}

MODEL_KEYS = ("arch", "n_layers", "d_model", "n_heads", "d_ffn", "vocab", "max_seq",
              "norm_eps", "rope_theta")

GEMM_SWEEP_KN = ((4096, 4096), (4096, 11008), (11008, 4096), (5120, 13824))
GEMM_SWEEP_M = (16, 128, 1024, 4096)


def model_cfg(name, **override):
    cfg = {k: CONFIGS[name][k] for k in MODEL_KEYS}
    cfg.update(override)
    return cfg


def linear_shapes(cfg):
    """(name, K, N) of the block linears in their fixed enumeration order."""
    d, f = cfg["d_model"], cfg["d_ffn"]
    if cfg["arch"] == "llama":
        return [("q", d, d), ("k", d, d), ("v", d, d), ("o", d, d),
                ("gate", d, f), ("up", d, f), ("down", f, d)]
    return [("q", d, d), ("k", d, d), ("v", d, d), ("o", d, d), ("fc1", d, f), ("fc2", f, d)]


def _gen(seed, device="cpu"):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal_fp32(shape, std, seed, device="cpu"):
    return torch.randn(shape, generator=_gen(seed, device), dtype=torch.float32,
                       device=device) * std


def raw_model_tensors(cfg, seed=1000, device="cpu"):
    """Un-quantised random-init tensors of a model, one seed per tensor.

    Returns dict: embed bf16 [V][d], lm_head bf16 [V][d], pos_embed bf16 (opt),
    final_norm_w/b fp32, layers = list of dict(norm*_w/b fp32,
    lin = {name: dict(w fp32 [K][N] ~ N(0, 0.02) [, bias fp32 [N]])}).
    Quantising the fp32 weights is the caller's job (oracle or library).
    """
    tid = [int(seed)]

    def nxt():
        tid[0] += 1
        return tid[0]

    d, V = cfg["d_model"], cfg["vocab"]
    out = {"cfg": dict(cfg)}
    out["embed"] = normal_fp32((V, d), 0.02, nxt(), device).bfloat16()
    out["lm_head"] = normal_fp32((V, d), 0.02, nxt(), device).bfloat16()
    opt = cfg["arch"] == "opt"
    if opt:
        out["pos_embed"] = normal_fp32((cfg["max_seq"], d), 0.02, nxt(), device).bfloat16()
    out["final_norm_w"] = torch.ones(d, dtype=torch.float32, device=device)
    if opt:
        out["final_norm_b"] = torch.zeros(d, dtype=torch.float32, device=device)
    layers = []
    for _ in range(cfg["n_layers"]):
        layer = {"norm1_w": torch.ones(d, device=device), "norm2_w": torch.ones(d, device=device)}
        if opt:
            layer["norm1_b"] = torch.zeros(d, device=device)
            layer["norm2_b"] = torch.zeros(d, device=device)
        lin = {}
        for name, K, N in linear_shapes(cfg):
            ent = {"w": normal_fp32((K, N), 0.02, nxt(), device)}
            if opt:
                ent["bias"] = normal_fp32((N,), 0.02, nxt(), device).bfloat16().float()
            lin[name] = ent
        layer["lin"] = lin
        layers.append(layer)
    out["layers"] = layers
    return out


def tokens_and_labels(cfg, batch, seq, seed=7):
    """Uniform-random token ids; labels = tokens shifted left, last position ignored (-100)."""
    tok = torch.randint(0, cfg["vocab"], (batch, seq), generator=_gen(seed), dtype=torch.int32)
    lab = torch.full((batch, seq), -100, dtype=torch.int32)
    lab[:, :-1] = tok[:, 1:]
    return tok, lab


def gemm_case(M, K, N, seed=0, device="cpu"):
    """Standalone GEMM sweep inputs: X bf16 ~ N(0,1) [M][K]; q int8 uniform in [-8,7] [K][N];
    scales bf16 uniform in [0.005, 0.02] [ceil(K/128)][N]."""
    g = _gen(seed, device)
    x = torch.randn((M, K), generator=g, dtype=torch.float32, device=device).bfloat16()
    q = torch.randint(-8, 8, (K, N), generator=g, dtype=torch.int8, device=device)
    G = (K + 127) // 128
    s = (torch.rand((G, N), generator=g, dtype=torch.float32, device=device) * 0.015
         + 0.005).bfloat16()
    return x, q, s


def table16_case(M, K, N, seed=0, device="cpu"):
    """Inputs of the block-scaled 16-entry-codebook GEMM (NF4-style storage): X bf16 ~ N(0,1) [M][K]; codes
    int8 uniform in [0,15] [K][N]; scales bf16 uniform in [0.01, 0.04] [ceil(K/64)][N] (absmax-like: the
    table lies in [-1, 1]); table = 16 increasing fp32 values in [-1, 1] drawn from the seed (sorted uniform
    draws with the end points pinned to -1 and 1), standing in for a trained or published codebook."""
    g = _gen(seed, device)
    x = torch.randn((M, K), generator=g, dtype=torch.float32, device=device).bfloat16()
    codes = torch.randint(0, 16, (K, N), generator=g, dtype=torch.int8, device=device)
    B = (K + 63) // 64
    s = (torch.rand((B, N), generator=g, dtype=torch.float32, device=device) * 0.03 + 0.01).bfloat16()
    t = torch.sort(torch.rand((16,), generator=g, dtype=torch.float32, device=device) * 2.0 - 1.0).values
    t[0], t[15] = -1.0, 1.0
    return x, codes, s, t
