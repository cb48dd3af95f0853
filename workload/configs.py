"""The five benchmark configurations: model shapes, corpus recipes and run parameters.

Data only.  Shapes follow the benchmark definition; seeds follow the convention
pool = 100+i, corpus = 200+i, prompts = 300+i, continuations = 400+i, weights = 0.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str              # "f32" or "bf16": storage type of weights, activations fed to GEMMs and KV
    tied: bool = True
    rope_base: float = 10000.0
    rms_eps: float = 1e-6
    init_std: float = 0.02

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def matmul_params(self) -> int:
        """Parameters of all GEMM weights (LM head counted once when tied)."""
        per_layer = (self.qkv_rows * self.d_model + self.d_model * self.q_dim
                     + 3 * self.d_ff * self.d_model)
        return self.n_layers * per_layer + self.vocab * self.d_model

    def kv_bytes_per_token(self) -> int:
        esz = 4 if self.dtype == "f32" else 2
        return 2 * self.n_layers * self.kv_dim * esz


@dataclass(frozen=True)
class CorpusRecipe:
    n_docs: int
    len_lo: int
    len_hi: int             # inclusive
    pool_size: int
    zipf_s: float
    insert_rate: float
    phrase_lo: int = 3
    phrase_hi: int = 8      # inclusive


@dataclass(frozen=True)
class RunConfig:
    index: int
    name: str
    model: ModelShape
    corpus: CorpusRecipe
    n_max: int
    k: int
    p_min: int
    batches: Tuple[int, ...]
    ks: Tuple[int, ...]
    prompt_len: int
    max_new: int
    page_size: int = 16
    lambda_num: int = 3
    lambda_den: int = 4
    n_merged_tokens: int = 0   # config 3: merged n-gram tokens appended to the vocabulary

    @property
    def seed_pool(self) -> int: return 100 + self.index
    @property
    def seed_corpus(self) -> int: return 200 + self.index
    @property
    def seed_prompts(self) -> int: return 300 + self.index
    @property
    def seed_cont(self) -> int: return 400 + self.index
    @property
    def seed_weights(self) -> int: return 0


_CFG0 = RunConfig(
    index=0, name="tiny-f32",
    model=ModelShape(2, 128, 4, 4, 32, 512, 512, "f32"),
    corpus=CorpusRecipe(2000, 16, 48, 200, 1.1, 0.15),
    n_max=3, k=4, p_min=2, batches=(1,), ks=(4,), prompt_len=32, max_new=64)

_CFG1 = RunConfig(
    index=1, name="slm-135m",
    model=ModelShape(30, 576, 9, 3, 64, 1536, 49152, "bf16"),
    corpus=CorpusRecipe(50000, 20, 120, 5000, 1.2, 0.15),
    n_max=4, k=5, p_min=5, batches=(1, 16), ks=(5,), prompt_len=256, max_new=128)

_CFG2 = RunConfig(
    index=2, name="0.5b",
    model=ModelShape(24, 896, 14, 2, 64, 4864, 151936, "bf16"),
    corpus=CorpusRecipe(200000, 20, 120, 5000, 1.2, 0.15),
    n_max=4, k=5, p_min=5, batches=(1, 8, 32), ks=(3, 5, 8), prompt_len=512, max_new=256)

_CFG3 = replace(_CFG2, index=3, name="0.5b-merged-vocab", batches=(16,), ks=(5,), n_merged_tokens=8192)

_CFG4 = RunConfig(
    index=4, name="1.5b",
    model=ModelShape(28, 1536, 12, 2, 128, 8960, 151936, "bf16"),
    corpus=CorpusRecipe(1000000, 20, 200, 20000, 1.1, 0.10),
    n_max=5, k=6, p_min=5, batches=(1, 64), ks=(6,), prompt_len=1024, max_new=512)

CONFIGS = (_CFG0, _CFG1, _CFG2, _CFG3, _CFG4)


def get(index: int) -> RunConfig:
    return CONFIGS[index]


def shrunk(cfg: RunConfig, *, n_layers=None, vocab=None, n_docs=None, d_ff=None) -> RunConfig:
    """A reduced copy of a configuration (same head geometry) for quick parity cases."""
    m = cfg.model
    m = replace(m, n_layers=n_layers or m.n_layers, vocab=vocab or m.vocab, d_ff=d_ff or m.d_ff)
    c = replace(cfg.corpus, n_docs=n_docs or cfg.corpus.n_docs)
    return replace(cfg, model=m, corpus=c)
