"""KV shapes and workload configurations (synthetic stand-ins for the paper's traces).

The paper measures on recorded coding-agent trajectories (Section 5.1) that are not
available here; the configurations below keep their structure (closed-loop agents that
resend an ever-growing prompt, lognormal growth, tool gaps that set the interleave).
"""
from __future__ import annotations

from dataclasses import dataclass, field


@dataclass(frozen=True)
class KVShape:
    """One rank's paged KV geometry.  A *piece* is one layer's K or V of one block."""
    num_layers: int
    kv_heads: int
    head_dim: int
    block_size: int
    elem_bytes: int = 2  # bf16

    @property
    def pieces_per_block(self) -> int:
        return 2 * self.num_layers

    @property
    def piece_bytes(self) -> int:
        return self.block_size * self.kv_heads * self.head_dim * self.elem_bytes

    @property
    def block_bytes(self) -> int:
        return self.pieces_per_block * self.piece_bytes

    @property
    def bytes_per_token(self) -> int:
        return self.block_bytes // self.block_size

    def tp_shard(self, tp: int) -> "KVShape":
        """One tensor-parallel rank's share: max(1, ceil(H_kv / TP)) KV heads of every layer."""
        heads = max(1, -(-self.kv_heads // tp))
        return KVShape(self.num_layers, heads, self.head_dim, self.block_size, self.elem_bytes)


SHAPES = {
    # 4 layers, 2 KV heads, head_dim 64, block 16: piece 4 KiB, block 32 KiB
    "tiny": KVShape(4, 2, 64, 16),
    # Qwen3-30B-A3B-shaped: 48 layers, 4 KV heads, head_dim 128, block 16: 96 KiB/token
    "qwen3_30b_a3b": KVShape(48, 4, 128, 16),
    # Llama-3-8B-shaped: 32 layers, 8 KV heads, head_dim 128, block 32: 128 KiB/token
    "llama3_8b": KVShape(32, 8, 128, 32),
}


@dataclass(frozen=True)
class TraceConfig:
    name: str
    shape: str
    seed: int
    agents: int
    turns: int
    first_prompt: int
    append_median: float
    append_sigma: float
    context_cap: int
    vocab: int = 151936
    # interleave: "round_robin" | "tool_gap" (closed loop, exponential tool latency) |
    # "poisson_start" (tool_gap plus Poisson agent arrivals)
    interleave: str = "round_robin"
    tool_gap_mean_ms: float = 5000.0
    start_gap_mean_ms: float = 1000.0
    gpu_blocks: int = 0
    host_blocks: int = 0          # 0: sized at run time (working-set estimate / sweep)
    policy: str = "write_all"
    kappa_blocks: int = 8
    shared_prefix_tokens: int = 0     # tokens of a system prompt that every agent starts with
    extra: dict = field(default_factory=dict)


GIB = 1 << 30

CONFIGS = {
    # C0: tiny bit-exact case
    "c0": TraceConfig("c0", "tiny", 0, 8, 12, 512, 200.0, 1.0, 2048,
                      interleave="round_robin", gpu_blocks=128, host_blocks=256),
    # sibling of C0 with a host tier large enough that restores happen
    "c0_big_tier": TraceConfig("c0_big_tier", "tiny", 0, 8, 12, 512, 200.0, 1.0, 2048,
                               interleave="round_robin", gpu_blocks=128, host_blocks=1024),
    # C2: 32 agents x 40 turns, tier capacity = the Eq. 5 working-set size (computed at run time)
    "c2": TraceConfig("c2", "qwen3_30b_a3b", 2, 32, 40, 4096, 1500.0, 1.2, 65536,
                      interleave="tool_gap",
                      gpu_blocks=(20 * GIB) // SHAPES["qwen3_30b_a3b"].block_bytes,
                      host_blocks=0),
    # C3: same trace as C2, fixed 32 GiB tier, both policies (kappa = 2048 tokens)
    "c3": TraceConfig("c3", "qwen3_30b_a3b", 2, 32, 40, 4096, 1500.0, 1.2, 65536,
                      interleave="tool_gap",
                      gpu_blocks=(20 * GIB) // SHAPES["qwen3_30b_a3b"].block_bytes,
                      host_blocks=(32 * GIB) // SHAPES["qwen3_30b_a3b"].block_bytes,
                      kappa_blocks=2048 // 16),
    # C4: 128 agents x 60 turns, Llama-3-8B shape, Poisson arrivals, tier swept
    "c4": TraceConfig("c4", "llama3_8b", 4, 128, 60, 8192, 2000.0, 1.3, 131072,
                      interleave="poisson_start", gpu_blocks=24576, host_blocks=0),
}
