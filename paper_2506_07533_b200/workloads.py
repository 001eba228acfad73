"""The synthetic workloads (shapes, expert mixes, routing-sharing groups) and their
algorithmic byte counts.  Pure bookkeeping: no tensor arithmetic here."""
from __future__ import annotations

from dataclasses import dataclass

SLOT_BYTES_PER_TOKEN = (96, 160, 288, 512)      # K+V bytes per token and kv head at 2/4/8/16 bit


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    d_in: int
    batch: int
    context: int
    chunk: int
    dtype: int            # 0 fp16, 1 bf16
    rs_group: int
    mix: tuple            # target share of chunks at 2/4/8/16 bit
    outlier_frac: float
    decode_steps: int = 1
    gated_router: bool = True

    @property
    def n_groups(self):
        return (self.n_layers + self.rs_group - 1) // self.rs_group

    @property
    def n_chunks(self):
        return self.context // self.chunk


WORKLOADS = {
    # tiny single layer, fp16, linear "1024 x 4" router, 4 fixed outlier key channels
    "cfg1": Workload("cfg1", 1, 8, 8, 1024, 1, 4096, 128, 0, 1, (0.25, 0.25, 0.25, 0.25), 0.0,
                     gated_router=False),
    # Llama-2-7B-shaped decode
    "cfg2": Workload("cfg2", 32, 32, 32, 4096, 1, 32768, 128, 1, 3, (0.10, 0.40, 0.40, 0.10), 0.01),
    # Llama-2-13B-shaped long context, sharing groups of 4, 16 decode steps
    "cfg3": Workload("cfg3", 40, 40, 40, 5120, 1, 65536, 128, 1, 4, (0.10, 0.40, 0.40, 0.10), 0.01,
                     decode_steps=16),
    # Llama-3-8B-shaped GQA, the 128k-context target
    "cfg4": Workload("cfg4", 32, 32, 8, 4096, 4, 131072, 256, 1, 3, (0.60, 0.30, 0.05, 0.05), 0.01),
    # prefill quantise+route sweep: one layer, 32 kv heads, 131072 tokens; the chunk size and the
    # map (forced uniform widths or router-chosen) are varied by the caller
    "cfg5": Workload("cfg5", 1, 32, 32, 4096, 1, 131072, 128, 1, 1, (0.25, 0.25, 0.25, 0.25), 0.01),
}


def cache_bytes_per_layer(counts, chunk: int, n_kv_heads: int, tail_len: int = 0) -> int:
    """Packed bytes of one layer: counts[b][w] chunks of width w for sequence b."""
    total = 0
    for row in counts:
        for w in range(4):
            total += int(row[w]) * chunk * SLOT_BYTES_PER_TOKEN[w] * n_kv_heads
        total += tail_len * 512 * n_kv_heads
    return total


def decode_bytes_per_layer(counts, wl: Workload, n_splits: int, tail_len: int = 0) -> int:
    """Algorithmic bytes of one decode-attention call: packed payload + scale/zero + tail,
    the query, the split partials (written, then read by the combine) and the output."""
    kv = cache_bytes_per_layer(counts, wl.chunk, wl.n_kv_heads, tail_len)
    q = wl.batch * wl.n_q_heads * 128 * 2
    partials = 2 * wl.batch * wl.n_q_heads * n_splits * 130 * 4
    out = wl.batch * wl.n_q_heads * 128 * 4
    return kv + q + partials + out


def quantize_bytes_per_layer(counts, wl: Workload, T: int) -> int:
    """K and V read once (512 B per token and head) plus the packed bytes written."""
    tail = T % wl.chunk
    return wl.batch * T * wl.n_kv_heads * 512 + cache_bytes_per_layer(counts, wl.chunk, wl.n_kv_heads, tail)


def route_bytes_per_group(wl: Workload, T: int, rf_first_chunk: bool = True) -> int:
    """Hidden rows of the routed chunks, read once."""
    chunks = T // wl.chunk - (1 if rf_first_chunk else 0)
    return wl.batch * max(chunks, 0) * wl.chunk * wl.d_in * 2
