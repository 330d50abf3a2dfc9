"""Model shapes and seeded random-init weight tables for the target DiT and the drafter.

Shapes follow the workloads the paper evaluates (DiT-XL/2 on 4x32x32 and 4x64x64
latents, Sec. 4) plus two small ones used for parity tests.  Weight values are
i.i.d. N(0, std^2): there are no trained checkpoints to stand in for.

Every linear layer is stored row-major as [out_features, in_features] and is
applied as y = W x + b.  Tensors that exist once per transformer block are
stacked over a leading `depth` axis.
"""
from dataclasses import dataclass
import numpy as np

from .rng import normal, round_to_bf16


@dataclass(frozen=True)
class DiTShape:
    name: str
    C: int = 4            # latent channels
    H: int = 32           # latent height
    W: int = 32           # latent width
    patch: int = 2
    D: int = 1152         # hidden width
    depth: int = 28
    heads: int = 16
    n_classes: int = 1000
    mlp_ratio: int = 4
    freq_dim: int = 256   # sinusoidal timestep features
    learn_sigma: bool = True   # output keeps 2C channels; only the first C are the noise prediction

    @property
    def n_tok(self) -> int:
        return (self.H // self.patch) * (self.W // self.patch)

    @property
    def d_head(self) -> int:
        return self.D // self.heads

    @property
    def c_out(self) -> int:
        return 2 * self.C if self.learn_sigma else self.C

    @property
    def patch_dim(self) -> int:
        return self.C * self.patch * self.patch

    @property
    def out_dim(self) -> int:
        return self.c_out * self.patch * self.patch

    @property
    def d_latent(self) -> int:
        return self.C * self.H * self.W

    def n_params(self) -> int:
        D, F = self.D, self.mlp_ratio * self.D
        per_block = (6 * D * D + 6 * D) + (3 * D * D + 3 * D) + (D * D + D) + (F * D + F) + (D * F + D)
        emb = (D * self.freq_dim + D) + (D * D + D) + (self.n_classes + 1) * D + (D * self.patch_dim + D)
        fin = (2 * D * D + 2 * D) + (self.out_dim * D + self.out_dim)
        return self.depth * per_block + emb + fin

    def drafter_params(self, n_blocks: int = 1) -> int:
        D, F = self.D, self.mlp_ratio * self.D
        per_block = (6 * D * D + 6 * D) + (3 * D * D + 3 * D) + (D * D + D) + (F * D + F) + (D * F + D)
        fc = D * 2 * D + D
        fin = (2 * D * D + 2 * D) + (self.out_dim * D + self.out_dim)
        return fc + n_blocks * per_block + fin

    def flops_per_sequence(self, depth=None) -> float:
        """Algorithmic FLOPs of one forward of one sequence: 2MNK per linear layer
        plus 4 * n_tok^2 * d_head per (head, block); nothing else is counted."""
        depth = self.depth if depth is None else depth
        D, F, T = self.D, self.mlp_ratio * self.D, self.n_tok
        gemm = 2.0 * T * (3 * D * D + D * D + 2 * F * D)
        attn = 4.0 * T * T * self.d_head * self.heads
        return depth * (gemm + attn)


TINY = DiTShape("tiny", H=8, W=8, D=64, depth=2, heads=2, n_classes=10)
DIT_S2 = DiTShape("DiT-S/2", H=32, W=32, D=384, depth=12, heads=6)
DIT_XL2_256 = DiTShape("DiT-XL/2-256", H=32, W=32)
DIT_XL2_512 = DiTShape("DiT-XL/2-512", H=64, W=64)


def pos_embed_2d(shape: DiTShape) -> np.ndarray:
    """Fixed 2-D sine/cosine position table [n_tok, D] (a constant weight of the model).

    The first D/2 features encode the patch row, the last D/2 the patch column;
    each half is [sin(p*w_i), cos(p*w_i)] with w_i = 10000^(-i/(D/4)).
    """
    gh, gw = shape.H // shape.patch, shape.W // shape.patch
    q = shape.D // 4
    w = 1.0 / (10000.0 ** (np.arange(q, dtype=np.float64) / q))
    rows, cols = np.meshgrid(np.arange(gh, dtype=np.float64), np.arange(gw, dtype=np.float64), indexing="ij")

    def enc(p):
        a = p.reshape(-1, 1) * w.reshape(1, -1)
        return np.concatenate([np.sin(a), np.cos(a)], axis=1)

    return np.concatenate([enc(rows), enc(cols)], axis=1).astype(np.float32)


def _mat(seed, stream, shape, std, bf16):
    a = normal(seed, stream, shape, std=std)
    return round_to_bf16(a) if bf16 else a


def _block_stack(seed, base, shape: DiTShape, depth, std, ada_std, bf16):
    D, F = shape.D, shape.mlp_ratio * shape.D
    w = {}
    w["ada_w"] = _mat(seed, base + 0, (depth, 6 * D, D), ada_std, bf16)
    w["ada_b"] = normal(seed, base + 1, (depth, 6 * D), std=ada_std)
    w["qkv_w"] = _mat(seed, base + 2, (depth, 3 * D, D), std, bf16)
    w["qkv_b"] = normal(seed, base + 3, (depth, 3 * D), std=std)
    w["proj_w"] = _mat(seed, base + 4, (depth, D, D), std, bf16)
    w["proj_b"] = normal(seed, base + 5, (depth, D), std=std)
    w["fc1_w"] = _mat(seed, base + 6, (depth, F, D), std, bf16)
    w["fc1_b"] = normal(seed, base + 7, (depth, F), std=std)
    w["fc2_w"] = _mat(seed, base + 8, (depth, D, F), std, bf16)
    w["fc2_b"] = normal(seed, base + 9, (depth, D), std=std)
    return w


def make_target_weights(shape: DiTShape, seed: int, bf16: bool = False, std: float = 0.02,
                        ada_std: float | None = None, out_gain: float = 1.0) -> dict:
    """Random-init target DiT.  `bf16=True` rounds every GEMM weight matrix to a
    bf16-representable value (biases, embeddings and the two narrow projections
    stay fp32).  `ada_std` sets the modulation layers' std (default: `std`);
    larger values make the gated branches contribute visibly to the output.
    `out_gain` scales the final projection so the size of the predicted noise
    can be moved between acceptance regimes."""
    ada_std = std if ada_std is None else ada_std
    D = shape.D
    w = {}
    w["t_w1"] = _mat(seed, 1, (D, shape.freq_dim), std, bf16)
    w["t_b1"] = normal(seed, 2, (D,), std=std)
    w["t_w2"] = _mat(seed, 3, (D, D), std, bf16)
    w["t_b2"] = normal(seed, 4, (D,), std=std)
    w["y_emb"] = normal(seed, 5, (shape.n_classes + 1, D), std=std)
    w["pe_w"] = normal(seed, 6, (D, shape.patch_dim), std=std)
    w["pe_b"] = normal(seed, 7, (D,), std=std)
    w["pos"] = pos_embed_2d(shape)
    w.update(_block_stack(seed, 100, shape, shape.depth, std, ada_std, bf16))
    w["fada_w"] = _mat(seed, 20, (2 * D, D), ada_std, bf16)
    w["fada_b"] = normal(seed, 21, (2 * D,), std=ada_std)
    w["fin_w"] = normal(seed, 22, (shape.out_dim, D), std=std * out_gain)
    w["fin_b"] = normal(seed, 23, (shape.out_dim,), std=std * out_gain)
    return w


def make_drafter_weights(shape: DiTShape, seed: int, n_blocks: int = 1, bf16: bool = False,
                         std: float = 0.02, ada_std: float | None = None, out_gain: float = 1.0) -> dict:
    """Random-init drafter: fusion layer [D, 2D], `n_blocks` transformer blocks and
    an output head of its own.  It has no embedding tables: it reuses the target's."""
    ada_std = std if ada_std is None else ada_std
    D = shape.D
    w = {}
    w["fc_w"] = _mat(seed, 1001, (D, 2 * D), std, bf16)
    w["fc_b"] = normal(seed, 1002, (D,), std=std)
    w.update(_block_stack(seed, 1100, shape, n_blocks, std, ada_std, bf16))
    w["fada_w"] = _mat(seed, 1020, (2 * D, D), ada_std, bf16)
    w["fada_b"] = normal(seed, 1021, (2 * D,), std=ada_std)
    w["fin_w"] = normal(seed, 1022, (shape.out_dim, D), std=std * out_gain)
    w["fin_b"] = normal(seed, 1023, (shape.out_dim,), std=std * out_gain)
    return w
