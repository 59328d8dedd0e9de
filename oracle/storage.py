"""Storage accounting of the HLQ format (test infrastructure).

With fp16 scales and zero-points (caption of the C4 perplexity table) a group
of G weights stores q bits per weight, q scales and one zero-point:

    bits per weight = q + 16 * (q + 1) / G

which the paper prints as 2.37 (q=2, G=128), 2.75 (q=2, G=64), 3.50 (q=3,
G=128); uniform quantisation stores one scale and one zero-point per group,
q + 32 / G (2.25, 3.25).  The model-size table counts every linear of every
transformer block as quantised and leaves the embedding and the output head
in fp16 (Appendix E), in units of 2^30 bytes.
"""

from __future__ import annotations


def hlq_bits_per_weight(q: int, G: int) -> float:
    return q + 16.0 * (q + 1) / G


def uniform_bits_per_weight(q: int, G: int) -> float:
    return q + 32.0 / G


def hlq_layer_bytes(q: int, G: int, N: int, K: int) -> int:
    """Exact bytes of one layer's bit-planes, scales and offsets."""
    if K % G:
        raise ValueError("K must be a multiple of G")
    return q * N * K // 8 + 2 * (q + 1) * N * (K // G)


def llama_block_weights(hidden: int, kv_dim: int, ffn: int) -> int:
    """Quantised weights of one LLaMA block: q,k,v,o projections + gate, up, down."""
    attn = hidden * hidden + 2 * kv_dim * hidden + hidden * hidden
    mlp = 3 * ffn * hidden
    return attn + mlp


def llama_model_gib(bits_per_weight: float, blocks: int, hidden: int, kv_dim: int,
                    ffn: int, vocab: int) -> float:
    """Model size in GiB: quantised blocks + fp16 embedding and output head."""
    quant = blocks * llama_block_weights(hidden, kv_dim, ffn) * bits_per_weight / 8.0
    fp16 = 2 * vocab * hidden * 2
    return (quant + fp16) / float(1 << 30)
