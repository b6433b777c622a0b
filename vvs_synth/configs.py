"""Model / workload shapes of the synthetic verify-step workloads.

Shapes only (no arithmetic of the method).  `CONFIGS` mirrors the five benchmark
configurations; the `*_small` entries are scaled-down versions with the same structure that
the CPU oracle finishes in seconds and that still span several kernel tiles plus a ragged
tail.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

ROPE_NONE, ROPE_1D, ROPE_2D_GRID = 0, 1, 2
DTYPE_FP32, DTYPE_BF16 = 0, 1
MODE_STRICT, MODE_RELAXED = 0, 1


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int              # V: image-codebook size = number of logits
    vocab_offset: int = 0   # first LM-head row of the image codebook
    lm_rows: int = 0        # total LM-head rows (>= vocab_offset + vocab); 0 -> vocab
    tok_rows: int = 0       # embedding-table rows; 0 -> lm_rows
    s_max: int = 640        # KV-cache capacity per sequence
    rope_mode: int = ROPE_NONE
    rope_grid_w: int = 0
    n_prefix: int = 0       # positions < n_prefix are prefix tokens (2-D rope: no rotation)
    rope_base: float = 10000.0
    rms_eps: float = 1e-5
    dtype: int = DTYPE_BF16

    def __post_init__(self):
        if self.lm_rows == 0:
            object.__setattr__(self, "lm_rows", self.vocab_offset + self.vocab)
        if self.tok_rows == 0:
            object.__setattr__(self, "tok_rows", self.lm_rows)

    @property
    def params_per_layer(self) -> int:
        d, ff = self.d_model, self.d_ff
        return 3 * d * d + d * d + 2 * ff * d + ff * d

    @property
    def streamed_params(self) -> int:
        """Weights a verify step must read once: all layers + the image slice of the LM head."""
        return self.n_layers * self.params_per_layer + self.vocab * self.d_model


TINY = ModelShape("tiny_fp32", 2, 256, 4, 64, 1024, 1024, s_max=128,
                  rope_mode=ROPE_1D, dtype=DTYPE_FP32)
XL = ModelShape("llamagen_xl", 36, 1280, 20, 64, 3456, 16384, s_max=592,
                rope_mode=ROPE_2D_GRID, rope_grid_w=24, n_prefix=1)
B7 = ModelShape("visual_ar_7b", 32, 4096, 32, 128, 11008, 8192, vocab_offset=32768,
                lm_rows=65536, s_max=2384, rope_mode=ROPE_1D, n_prefix=64)

# Structure-preserving reductions for CPU-time-bounded parity tests.
XL_SMALL = replace(XL, name="llamagen_xl_small", n_layers=3, d_model=320, n_heads=5,
                   d_ff=864, vocab=2048 + 128 + 40, lm_rows=0, tok_rows=0, s_max=592)
B7_SMALL = replace(B7, name="visual_ar_7b_small", n_layers=2, d_model=512, n_heads=4,
                   d_ff=1376, vocab=1024 + 72, vocab_offset=512, lm_rows=4096, tok_rows=0,
                   s_max=400)


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    n_images: int           # B
    n_cfg: int              # C: 2 = cond + uncond rows with guidance, 1 = no guidance
    cfg_scale: float
    n_draft_max: int        # K
    n_forced: int = 1       # F
    fill_lo: int = 1
    fill_hi: int = 575      # cache fill L ~ U{fill_lo..fill_hi} per image
    mode: int = MODE_STRICT
    nbr_k: int = 1
    delta: float = float("inf")
    temperature: float = 1.0
    latent_dim: int = 8
    q_noise_std: float = 1.0   # draft logits = target logits + N(0, q_noise_std^2)
    seed: int = 0x56565300

    @property
    def n_rows(self) -> int:
        return self.n_images * self.n_cfg

    @property
    def block_len(self) -> int:
        return self.n_forced + self.n_draft_max


CONFIGS = {
    0: Workload("tiny_fp32_strict", TINY, 1, 1, 1.0, 4, fill_lo=64, fill_hi=64,
                q_noise_std=2.0, seed=0x56565300),
    1: Workload("xl_bf16_cfg_b1_k8", XL, 1, 2, 2.0, 8, seed=0x56565301),
    2: Workload("xl_bf16_cfg_b16_k8_relaxed", XL, 16, 2, 2.0, 8, mode=MODE_RELAXED, nbr_k=64,
                seed=0x56565302),
    3: Workload("7b_bf16_cfg_b1_k8", B7, 1, 2, 2.0, 8, fill_lo=1500, fill_hi=1500,
                seed=0x56565303),
}
