"""Model shapes and workloads of the synthetic stand-ins for the paper's models.

The paper evaluates Ouro (R=4) and Raven (R=32) checkpoints on public
benchmarks (Sec. 6, App. A); neither the checkpoints nor the datasets are
available offline, so random weights of the same shapes and uniform-random
prompts of the same lengths stand in for them.
"""
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ModelShape:
    name: str
    vocab: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    n_recurrent: int          # layers in the shared stack B
    R: int                    # recurrences
    weight_dtype: str         # "fp32" | "bf16"
    tied: bool                # lm_head shares the embedding matrix
    n_prelude: int = 0
    n_coda: int = 0
    rms_eps: float = 1e-6
    rope_theta: float = 10000.0
    std: float = 0.02         # N(0, std) for every matrix
    out_scale: float = 0.3    # multiplies W_o and W_down after drawing

    def n_params(self) -> int:
        h, f = self.hidden, self.ffn
        qkv = (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim * h
        per_layer = qkv + self.n_q_heads * self.head_dim * h + 3 * f * h + 2 * h
        n = self.vocab * h * (1 if self.tied else 2) + h
        return n + per_layer * (self.n_prelude + self.n_recurrent + self.n_coda)

    def with_(self, **kw) -> "ModelShape":
        return replace(self, **kw)


@dataclass(frozen=True)
class Workload:
    name: str
    model: str
    prompt_len: int
    decode_len: int
    temperature: float        # 0 = greedy
    d1: int
    d2: int                   # 0 = single proposal
    gate: bool = True
    batch: int = 1
    prompt_seed: int = 1
    sample_seed: int = 2
    weight_seed: int = 0
    top_k: int = 0            # filters of the readout (0 / 1.0 = off); only used when temperature > 0
    top_p: float = 1.0


CONFIGS = {
    # config 0: tiny looped LM, fp32, tied head
    "tiny": ModelShape("tiny", vocab=512, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                       ffn=688, n_recurrent=2, R=4, weight_dtype="fp32", tied=True),
    # the same tiny widths with bf16 weights and an untied head (exercises the tensor-core path
    # and, because it drafts badly, the rejection / rollback paths)
    "tiny_bf16": ModelShape("tiny_bf16", vocab=512, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                            ffn=704, n_recurrent=2, R=4, weight_dtype="bf16", tied=False),
    # grouped-query attention, the head layout of the Raven-style config (4 query heads per KV head, head size 64)
    "tiny_gqa": ModelShape("tiny_gqa", vocab=512, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=64,
                           ffn=1024, n_recurrent=2, R=4, weight_dtype="bf16", tied=False),
    # and with head size 128, fp32 weights
    "tiny_gqa_f32": ModelShape("tiny_gqa_f32", vocab=512, hidden=512, n_q_heads=4, n_kv_heads=1, head_dim=128,
                               ffn=1024, n_recurrent=2, R=4, weight_dtype="fp32", tied=True),
    # deeper loops (the Raven-style models run R = 32): more pipeline levels in flight, larger branch bounds
    "tiny_r8": ModelShape("tiny_r8", vocab=512, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                          ffn=704, n_recurrent=2, R=8, weight_dtype="bf16", tied=False),
    "tiny_r16": ModelShape("tiny_r16", vocab=512, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                           ffn=704, n_recurrent=1, R=16, weight_dtype="bf16", tied=False),
    # the Raven family's loop count: R = 32, where (d1, d2) = (2, 8) allows up to 249 branches in a pass (Sec. 4.3)
    "tiny_r32": ModelShape("tiny_r32", vocab=512, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                           ffn=704, n_recurrent=1, R=32, weight_dtype="bf16", tied=False),
    "tiny_raven_r32": ModelShape("tiny_raven_r32", vocab=512, hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=64,
                                 ffn=704, n_recurrent=1, R=32, weight_dtype="bf16", tied=False, n_prelude=1, n_coda=1),
    # a mid-size bf16 model whose GEMMs span several tiles, K-slices and a ragged last tile
    "small_bf16": ModelShape("small_bf16", vocab=4000, hidden=768, n_q_heads=6, n_kv_heads=6, head_dim=128,
                             ffn=2000, n_recurrent=3, R=4, weight_dtype="bf16", tied=False),
    # Raven layout at test size: prelude and coda blocks around the recurrent block, an adapter on [state; prelude output],
    # grouped-query attention with head size 64 (the head layout of the Raven-style benchmark config), R = 16
    "tiny_raven": ModelShape("tiny_raven", vocab=512, hidden=256, n_q_heads=8, n_kv_heads=2, head_dim=64,
                             ffn=704, n_recurrent=2, R=16, weight_dtype="bf16", tied=False, n_prelude=1, n_coda=1),
    "tiny_raven_r4": ModelShape("tiny_raven_r4", vocab=512, hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64,
                                ffn=704, n_recurrent=2, R=4, weight_dtype="bf16", tied=False, n_prelude=2, n_coda=2),
    # config 1: Ouro-1.4B shape
    "ouro_1p4b": ModelShape("ouro_1p4b", vocab=49152, hidden=2048, n_q_heads=16, n_kv_heads=16, head_dim=128,
                            ffn=5632, n_recurrent=24, R=4, weight_dtype="bf16", tied=False),
    # config 2: Ouro-2.6B shape
    "ouro_2p6b": ModelShape("ouro_2p6b", vocab=49152, hidden=2048, n_q_heads=16, n_kv_heads=16, head_dim=128,
                            ffn=5632, n_recurrent=48, R=4, weight_dtype="bf16", tied=False),
    # config 4: Raven-style prelude / recurrent / coda model
    "raven": ModelShape("raven", vocab=128256, hidden=2048, n_q_heads=32, n_kv_heads=8, head_dim=64,
                        ffn=8192, n_recurrent=4, R=16, weight_dtype="bf16", tied=False, n_prelude=2, n_coda=2),
}

WORKLOADS = {
    "tiny": Workload("tiny", "tiny", prompt_len=16, decode_len=64, temperature=0.0, d1=1, d2=0),
    "ouro_1p4b": Workload("ouro_1p4b", "ouro_1p4b", prompt_len=512, decode_len=512, temperature=0.0, d1=1, d2=2),
    "ouro_2p6b": Workload("ouro_2p6b", "ouro_2p6b", prompt_len=1024, decode_len=1024, temperature=1.0, d1=1, d2=2),
    # the paper's sampling setting for its reasoning models (Sec. 6 "Models and Evaluations": T = 1.0, top-p 0.7) on the headline shape
    "ouro_1p4b_top_p": Workload("ouro_1p4b_top_p", "ouro_1p4b", prompt_len=512, decode_len=512, temperature=1.0, d1=1,
                                d2=2, top_p=0.7),
    "raven": Workload("raven", "raven", prompt_len=256, decode_len=512, temperature=0.0, d1=2, d2=8),
    "kv_bound": Workload("kv_bound", "ouro_1p4b", prompt_len=8192, decode_len=256, temperature=0.7, d1=1, d2=2,
                         batch=8),
}


def get_config(name: str) -> ModelShape:
    return CONFIGS[name]
