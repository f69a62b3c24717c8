"""Model shapes and workload recipes used by the tests and the benchmark."""
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ModelShape:
    """Shape of a Qwen3-style decoder (the base model the paper fine-tunes, Section 3.1)."""
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    intermediate: int
    vocab: int
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6
    dtype: str = "bf16"          # storage type of the weights: "f32" or "bf16"

    def with_(self, **kw):
        return replace(self, **kw)

    @property
    def q_dim(self):
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self):
        return self.n_kv_heads * self.head_dim

    @property
    def params_per_layer(self):
        h, i = self.hidden, self.intermediate
        return (h * (self.q_dim + 2 * self.kv_dim) + self.q_dim * h + 3 * h * i
                + 2 * h + 2 * self.head_dim)


SHAPES = {
    # Smallest case: the oracle finishes it in well under a second.
    "tiny": ModelShape(n_layers=4, hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64,
                       intermediate=768, vocab=1024, dtype="f32"),
    # Same layer geometry as the 4B shape (head_dim 128, 4 query heads per KV head,
    # K extents that are not powers of two) but small enough for element-by-element
    # parity in seconds; vocab is not a multiple of the row tile of the head kernel.
    "mid": ModelShape(n_layers=6, hidden=640, n_q_heads=8, n_kv_heads=2, head_dim=128,
                      intermediate=1824, vocab=5000, dtype="bf16"),
    # The paper's default base model (Section 3.1): 36 layers, last 8 are decoding layers.
    "qwen3_4b": ModelShape(n_layers=36, hidden=2560, n_q_heads=32, n_kv_heads=8, head_dim=128,
                           intermediate=9728, vocab=151936, dtype="bf16"),
    # The same layer and head geometry with 4 layers: small enough (1.6 GB) to capture with a
    # profiler, large enough that every launch streams far more than the L2 holds.
    "qwen3_4b_l4": ModelShape(n_layers=4, hidden=2560, n_q_heads=32, n_kv_heads=8, head_dim=128,
                              intermediate=9728, vocab=151936, dtype="bf16"),
}


@dataclass(frozen=True)
class Workload:
    """One decode workload: model shape, DMTD split and cycle, batch, prompt and output length."""
    name: str
    shape: str
    L_d: int
    tau: int
    batch: int
    prompt_len: int
    gen_len: int
    weight_seed: int = 0
    prompt_seed: int = 1
    kv_dtype: str = "bf16"       # storage type of the KV cache: "f32", "bf16" or "f16"


WORKLOADS = {
    # Stand-ins for the paper's throughput study (Section 3.4: random-vocabulary prompts of a
    # static length, fixed generation length); sizes follow the build's baseline configs.
    "tiny_b1": Workload("tiny_b1", "tiny", L_d=2, tau=3, batch=1, prompt_len=32, gen_len=24),
    # KV cache type: a bf16 cache alone moves the logits of the 36-layer model by more than the logit
    # tolerance, so the workloads whose logits are held to it use fp16 (half of fp32's bytes, tensor-core
    # attention, 7e-3 on the logits at full depth; an fp32 cache gives 2e-4 and is what the remaining
    # tests use); bf16 where the workload says so.
    "qwen3_4b_b1": Workload("qwen3_4b_b1", "qwen3_4b", L_d=8, tau=3, batch=1, prompt_len=512,
                            gen_len=256, kv_dtype="f16"),
    "qwen3_4b_l4_b1": Workload("qwen3_4b_l4_b1", "qwen3_4b_l4", L_d=2, tau=3, batch=1, prompt_len=512,
                               gen_len=64, kv_dtype="f16"),
    "qwen3_4b_b32": Workload("qwen3_4b_b32", "qwen3_4b", L_d=8, tau=3, batch=32, prompt_len=1024,
                             gen_len=512, kv_dtype="f16"),
    # the same batch on the 4-layer model: small enough to list every launch under a profiler
    "qwen3_4b_l4_b32": Workload("qwen3_4b_l4_b32", "qwen3_4b_l4", L_d=2, tau=3, batch=32, prompt_len=1024,
                                gen_len=48, kv_dtype="f16"),
    "qwen3_4b_long": Workload("qwen3_4b_long", "qwen3_4b", L_d=8, tau=3, batch=8,
                              prompt_len=16384, gen_len=256),
}
