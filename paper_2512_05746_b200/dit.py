"""Layer list of the quantized linears of a DiT-style diffusion transformer (shapes only, no arithmetic).

The second network family the method is evaluated on is a transformer over latent patches: `depth` identical
blocks of width `hidden`, each with a conditioning (adaLN modulation) linear on the per-sample embedding, the
attention QKV and output projections, and a two-layer MLP with ratio 4; in front of them the two-layer timestep
embedding MLP, after them the modulation of the final layer.  The patch embedding and the final projection are
the first / last layers and stay unquantized.  Width 1152 = 9 x 128, so the Hadamard matrix is block-diagonal
with 128-point blocks.
"""
from __future__ import annotations


def quantized_layers(batch: int = 32, tokens: int = 256, hidden: int = 1152, depth: int = 28, mlp_ratio: int = 4,
                     freq_dim: int = 256, had_block: int = 128) -> list[dict]:
    """One dict per quantized linear, in execution order: kind 'linear', M, K, N, had_block, macs, name."""
    layers: list[dict] = []

    def linear(name, M, K, N):
        layers.append(dict(kind="linear", name=name, M=M, K=K, N=N, had_block=min(had_block, K), macs=M * N * K))

    M = batch * tokens
    linear("t_embedder.0", batch, freq_dim, hidden)
    linear("t_embedder.2", batch, hidden, hidden)
    for b in range(depth):
        linear(f"block{b}.adaLN", batch, hidden, 6 * hidden)
        linear(f"block{b}.qkv", M, hidden, 3 * hidden)
        linear(f"block{b}.proj", M, hidden, hidden)
        linear(f"block{b}.fc1", M, hidden, mlp_ratio * hidden)
        linear(f"block{b}.fc2", M, mlp_ratio * hidden, hidden)
    linear("final.adaLN", batch, hidden, 2 * hidden)
    return layers
