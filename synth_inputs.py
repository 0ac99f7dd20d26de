"""Seeded synthetic inputs for the integerized ViT matmul path.

This module only *draws data and parameters*: Gaussian tensors with the shapes of
ViT-Tiny/Small/Base blocks, outlier channels, and the step sizes that both the CPU oracle and the CUDA library receive as
plain inputs.  It performs none of the method's steps (no quantizer, no integer
contraction, no softmax) and imports neither implementation, so the two stay
independent while seeing bit-identical inputs.

The inputs stand in for the CIFAR-10 / DeiT-S workload of the paper's Section V,
which is not available offline; only shapes and value distributions are kept.

Random numbers: splitmix64 used as a counter-based generator (element i of a
stream is mix(seed + (i+1)*gamma)), turned into normals by Box-Muller in fp64
and rounded once to fp32.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
BASE_SEED = 250418547


def splitmix64(seed: int, n: int, start: int = 0) -> np.ndarray:
    """n outputs of splitmix64 seeded with `seed`, beginning at draw `start`."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + n + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GAMMA
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def substream(seed: int, tag: str) -> int:
    """A derived seed for a named tensor, so tensors do not share draws."""
    h = seed & 0xFFFFFFFFFFFFFFFF
    for ch in tag.encode():
        h = int(splitmix64(h ^ ch, 1)[0])
    return h


def uniform01(seed: int, n: int) -> np.ndarray:
    """fp64 uniforms in [0, 1) with 53 random bits."""
    return (splitmix64(seed, n) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def normal(seed: int, shape, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """fp32 normals (Box-Muller evaluated in fp64, rounded once)."""
    n = int(np.prod(shape))
    half = (n + 1) // 2
    u = uniform01(seed, 2 * half)
    u1 = 1.0 - u[:half]          # (0, 1]
    u2 = u[half:]
    r = np.sqrt(-2.0 * np.log(u1))
    z = np.concatenate([r * np.cos(2.0 * np.pi * u2), r * np.sin(2.0 * np.pi * u2)])[:n]
    return (mean + std * z).astype(np.float32).reshape(shape)


def choice_without_replacement(seed: int, n: int, k: int) -> np.ndarray:
    """k distinct indices in [0, n), by sorting n random keys."""
    keys = splitmix64(seed, n)
    return np.sort(np.argsort(keys, kind="stable")[:k])


# ---------------------------------------------------------------------------
# integer ranges and step sizes (parameters handed to both implementations)
# ---------------------------------------------------------------------------

def code_range(bits: int, signed: bool) -> tuple[int, int]:
    if signed:
        return -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    return 0, (1 << bits) - 1


def lsq_step(x: np.ndarray, bits: int, signed: bool) -> np.float32:
    """Per-tensor LSQ initialisation 2*mean|x|/sqrt(Qp), fp64 then one rounding."""
    qp = code_range(bits, signed)[1]
    s = 2.0 * float(np.mean(np.abs(x.astype(np.float64)))) / math.sqrt(qp)
    return np.float32(max(s, 1e-8))


def lsq_step_rows(w: np.ndarray, bits: int, signed: bool = True) -> np.ndarray:
    """Per-output-channel (row) LSQ initialisation for a weight matrix [N, K]."""
    qp = code_range(bits, signed)[1]
    s = 2.0 * np.mean(np.abs(w.astype(np.float64)), axis=1) / math.sqrt(qp)
    return np.maximum(s, 1e-8).astype(np.float32)


def gaussian_lsq_step(sigma: float, bits: int, signed: bool = True) -> np.float32:
    """LSQ initialisation for a N(0, sigma^2) tensor in closed form (E|x| = sigma*sqrt(2/pi))."""
    qp = code_range(bits, signed)[1]
    return np.float32(2.0 * sigma * math.sqrt(2.0 / math.pi) / math.sqrt(qp))


def gelu_lsq_step(sigma: float, bits: int, seed: int) -> np.float32:
    """LSQ initialisation for GELU(N(0, sigma^2)) from a 64k-sample Monte-Carlo mean."""
    from scipy.special import erf  # data statistics only
    y = normal(seed, (65536,), 0.0, sigma).astype(np.float64)
    g = 0.5 * y * (1.0 + erf(y / math.sqrt(2.0)))
    qp = code_range(bits, False)[1]
    return np.float32(2.0 * float(np.mean(np.abs(g))) / math.sqrt(qp))


# ---------------------------------------------------------------------------
# workload configurations
# ---------------------------------------------------------------------------

@dataclass(frozen=True)
class BlockConfig:
    name: str
    batch: int
    tokens: int
    dim: int
    heads: int
    bits: int = 4
    mlp_dim: int = 0           # 0: attention block only
    layers: int = 1
    outlier_frac: float = 0.0
    seed_index: int = 0
    head_dim: int = field(default=64)
    w_std: float = 0.02        # weight spread; larger values give peaked attention rows

    @property
    def rows(self) -> int:
        return self.batch * self.tokens

    @property
    def seed(self) -> int:
        return BASE_SEED + self.seed_index

    def with_(self, **kw) -> "BlockConfig":
        d = self.__dict__.copy()
        d.update(kw)
        return BlockConfig(**d)


VIT_TINY_BLOCK = BlockConfig("vit_tiny_attn_b1", 1, 197, 192, 3, 4, seed_index=1)
VIT_SMALL_BLOCK = BlockConfig("vit_small_attn_b64", 64, 197, 384, 6, 4, outlier_frac=0.01, seed_index=2)
VIT_BASE_LAYER = BlockConfig("vit_base_layer_b128", 128, 197, 768, 12, 4, mlp_dim=3072, seed_index=3)
VIT_BASE_ENCODER = BlockConfig("vit_base_12layer_b256", 256, 197, 768, 12, 4, mlp_dim=3072, layers=12, seed_index=4)
# The self-attention module of the paper's power table: DeiT-S width, 198 tokens (class + distillation + 196
# patches), 3-bit, with a LayerNorm over each head's 64 channels in front of the Q and K quantizers.
DEIT_S_ATTENTION = BlockConfig("deit_s_attn_n198_b64", 64, 198, 384, 6, 3, seed_index=5)
# The whole DeiT-S model the paper evaluates (Section V-A): 16x16x3 patches -> 384 channels, class and distillation
# tokens (198 tokens), 12 encoder layers with a 1536-wide MLP, final LayerNorm, two classifier heads (10 classes).
DEIT_S_MODEL = BlockConfig("deit_s_model_n198_b128", 128, 198, 384, 6, 4, mlp_dim=1536, layers=12, seed_index=6)
PATCH_DIM = 16 * 16 * 3
NUM_CLASSES = 10
CONFIGS = {c.name: c for c in (VIT_TINY_BLOCK, VIT_SMALL_BLOCK, VIT_BASE_LAYER, VIT_BASE_ENCODER, DEIT_S_ATTENTION,
                               DEIT_S_MODEL)}


def activations(cfg: BlockConfig, batch: int | None = None, first_image: int = 0) -> np.ndarray:
    """fp32 activations [batch*tokens, dim] ~ N(0,1); a seeded 1% of channels scaled x10 when asked.

    Images are drawn from per-image streams, so a subset of images of a large
    batch can be produced without generating the rest.
    """
    b = cfg.batch if batch is None else batch
    out = np.empty((b * cfg.tokens, cfg.dim), dtype=np.float32)
    for i in range(b):
        s = substream(cfg.seed, f"x/{first_image + i}")
        out[i * cfg.tokens:(i + 1) * cfg.tokens] = normal(s, (cfg.tokens, cfg.dim))
    if cfg.outlier_frac > 0.0:
        k = int(math.ceil(cfg.outlier_frac * cfg.dim))
        ch = choice_without_replacement(substream(cfg.seed, "outliers"), cfg.dim, k)
        out[:, ch] *= np.float32(10.0)
    return out


def outlier_channels(cfg: BlockConfig) -> np.ndarray:
    if cfg.outlier_frac <= 0.0:
        return np.zeros((0,), dtype=np.int64)
    k = int(math.ceil(cfg.outlier_frac * cfg.dim))
    return choice_without_replacement(substream(cfg.seed, "outliers"), cfg.dim, k)


def layer_parameters(cfg: BlockConfig, layer: int = 0) -> dict:
    """Random-init fp32 weights/biases of one block and every step size the path needs.

    Weights ~ N(0, 0.02), biases ~ N(0, 0.01), LayerNorm gamma ~ N(1, 0.02), beta ~ N(0, 0.02).
    Activation steps are LSQ initialisations derived from the *expected* Gaussian
    statistics of each tensor (closed form), so no implementation is needed to make them.
    """
    D, F, b = cfg.dim, cfg.mlp_dim, cfg.bits
    sd = lambda tag: substream(cfg.seed, f"L{layer}/{tag}")
    p: dict = {}
    ws = cfg.w_std
    p["w_qkv"] = normal(sd("w_qkv"), (3 * D, D), 0.0, ws)
    p["b_qkv"] = normal(sd("b_qkv"), (3 * D,), 0.0, 0.01)
    p["w_proj"] = normal(sd("w_proj"), (D, D), 0.0, ws)
    p["b_proj"] = normal(sd("b_proj"), (D,), 0.0, 0.01)
    p["s_w_qkv"] = lsq_step_rows(p["w_qkv"], b)
    p["s_w_proj"] = lsq_step_rows(p["w_proj"], b)
    # expected spread of the tensors along the path (unit-variance block input)
    x_rms = math.sqrt(1.0 + 99.0 * (math.ceil(cfg.outlier_frac * D) / D if cfg.outlier_frac > 0 else 0.0))
    sig_qkv = ws * math.sqrt(D) * x_rms
    p["s_x"] = gaussian_lsq_step(x_rms, b)          # used when the block input is not given explicitly
    p["s_q"] = gaussian_lsq_step(sig_qkv, b)
    p["s_k"] = gaussian_lsq_step(sig_qkv, b)
    p["s_v"] = gaussian_lsq_step(sig_qkv, b)
    qp_u = code_range(b, False)[1]
    p["s_p"] = np.float32(2.0 / (cfg.tokens * math.sqrt(qp_u)))       # mean|p| = 1/T exactly
    p["s_o"] = gaussian_lsq_step(1.2 * sig_qkv / math.sqrt(cfg.tokens) + 0.01, b)
    p["s_out"] = gaussian_lsq_step(ws * math.sqrt(D) * sig_qkv / math.sqrt(cfg.tokens) + 0.02, b)
    if F:
        p["ln1_g"] = normal(sd("ln1_g"), (D,), 1.0, 0.02)
        p["ln1_b"] = normal(sd("ln1_b"), (D,), 0.0, 0.02)
        p["ln2_g"] = normal(sd("ln2_g"), (D,), 1.0, 0.02)
        p["ln2_b"] = normal(sd("ln2_b"), (D,), 0.0, 0.02)
        p["w_fc1"] = normal(sd("w_fc1"), (F, D), 0.0, ws)
        p["b_fc1"] = normal(sd("b_fc1"), (F,), 0.0, 0.01)
        p["w_fc2"] = normal(sd("w_fc2"), (D, F), 0.0, ws)
        p["b_fc2"] = normal(sd("b_fc2"), (D,), 0.0, 0.01)
        p["s_w_fc1"] = lsq_step_rows(p["w_fc1"], b)
        p["s_w_fc2"] = lsq_step_rows(p["w_fc2"], b)
        p["s_ln"] = gaussian_lsq_step(1.0, b)
        p["s_g"] = gelu_lsq_step(ws * math.sqrt(D), b, sd("gelu_mc"))
    return p


def patch_rows(cfg: BlockConfig, batch: int | None = None, first_image: int = 0) -> np.ndarray:
    """Flattened, normalised image patches ~ N(0,1), fp32 [batch*tokens, PATCH_DIM].  The rows of the class and
    distillation tokens (the first two of every image) are zero: their embeddings come from the token table."""
    b = cfg.batch if batch is None else batch
    out = np.zeros((b * cfg.tokens, PATCH_DIM), dtype=np.float32)
    for i in range(b):
        s = substream(cfg.seed, f"patches/{first_image + i}")
        out[i * cfg.tokens + 2:(i + 1) * cfg.tokens] = normal(s, (cfg.tokens - 2, PATCH_DIM))
    return out


def model_end_parameters(cfg: BlockConfig) -> dict:
    """Random-init parameters of the model's two ends: patch embedding (a linear layer over flattened patches),
    the token table (class / distillation token and position embeddings, one fp32 row per token, added after the
    patch embedding), final LayerNorm, and the two classifier heads whose logits are summed."""
    sd = lambda tag: substream(cfg.seed, f"ends/{tag}")
    D, b = cfg.dim, cfg.bits
    p = {"w_pe": normal(sd("w_pe"), (D, PATCH_DIM), 0.0, cfg.w_std), "b_pe": normal(sd("b_pe"), (D,), 0.0, 0.01),
         "tokens": normal(sd("tokens"), (cfg.tokens, D), 0.0, 0.02),
         "lnf_g": normal(sd("lnf_g"), (D,), 1.0, 0.02), "lnf_b": normal(sd("lnf_b"), (D,), 0.0, 0.02),
         "w_head": normal(sd("w_head"), (NUM_CLASSES, D), 0.0, cfg.w_std),
         "b_head": normal(sd("b_head"), (NUM_CLASSES,), 0.0, 0.01),
         "w_head_dist": normal(sd("w_head_dist"), (NUM_CLASSES, D), 0.0, cfg.w_std),
         "b_head_dist": normal(sd("b_head_dist"), (NUM_CLASSES,), 0.0, 0.01)}
    for n in ("w_pe", "w_head", "w_head_dist"):
        p["s_" + n] = lsq_step_rows(p[n], b)
    p["s_patch"] = gaussian_lsq_step(1.0, b)
    p["s_lnf"] = gaussian_lsq_step(1.0, b)
    return p


def qk_norm_parameters(cfg: BlockConfig, layer: int = 0) -> dict:
    """Parameters of the per-head LayerNorm in front of the Q and K quantizers (gain ~ N(1, 0.02), offset
    ~ N(0, 0.02) over the head's channels, shared by the heads) and the step of the normalised values."""
    sd = lambda tag: substream(cfg.seed, f"L{layer}/{tag}")
    d = cfg.head_dim
    return {"qn_g": normal(sd("qn_g"), (d,), 1.0, 0.02), "qn_b": normal(sd("qn_b"), (d,), 0.0, 0.02),
            "kn_g": normal(sd("kn_g"), (d,), 1.0, 0.02), "kn_b": normal(sd("kn_b"), (d,), 0.0, 0.02),
            "s_qn": gaussian_lsq_step(1.0, cfg.bits), "s_kn": gaussian_lsq_step(1.0, cfg.bits)}


# ---------------------------------------------------------------------------
# operation / byte counts used by the benchmark reporter
# ---------------------------------------------------------------------------

def mac_counts(tokens: int, dim: int, heads: int, head_dim: int = 64, mlp_dim: int = 0) -> dict:
    """Multiply-accumulates per image of each integer contraction of one block."""
    T, D = tokens, dim
    c = {
        "qkv": T * D * 3 * D,
        "qk": heads * T * T * head_dim,
        "pv": heads * T * T * head_dim,
        "proj": T * D * D,
    }
    if mlp_dim:
        c["fc1"] = T * D * mlp_dim
        c["fc2"] = T * mlp_dim * D
    c["total"] = sum(c.values())
    return c


def head_mac_counts(n_tokens: int, in_dim: int, out_dim: int) -> dict:
    """Per-head counts in the notation of the paper's Table I (I, O, N)."""
    return {
        "linear_pe": in_dim * out_dim,
        "linear_mac": n_tokens * in_dim * out_dim,
        "matmul_qk_pe": n_tokens * n_tokens,
        "matmul_qk_mac": n_tokens * n_tokens * out_dim,
        "matmul_pv_pe": n_tokens * out_dim,
        "matmul_pv_mac": n_tokens * n_tokens * out_dim,
        "layernorm_pe": 2 * out_dim,
        "layernorm_mac": 2 * n_tokens * out_dim,
        "delay": n_tokens * out_dim,
    }
