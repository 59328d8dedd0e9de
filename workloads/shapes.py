"""Layer shapes and call lists of the benchmark configurations.

Shapes are the LLaMA-3.1 8B / 70B linear layers with q/k/v and gate/up merged
(out-features N, in-features K).  A "call" is one (name, M, N, K, q, G) tuple.
"""

from __future__ import annotations

from dataclasses import dataclass

# (N, K) per merged linear
LLAMA31_8B = {
    "qkv": (6144, 4096),
    "o": (4096, 4096),
    "gate_up": (28672, 4096),
    "down": (4096, 14336),
}
LLAMA31_70B = {
    "qkv": (10240, 8192),
    "o": (8192, 8192),
    "gate_up": (57344, 8192),
    "down": (8192, 28672),
}


@dataclass(frozen=True)
class Call:
    name: str
    M: int
    N: int
    K: int
    q: int
    G: int = 128
    outliers: bool = False

    @property
    def tag(self) -> str:
        return f"{self.name}/q{self.q}/G{self.G}/{self.N}x{self.K}"


def algorithmic_bytes(M: int, N: int, K: int, q: int, G: int) -> int:
    """Bytes one call must move: bit-planes + fp16 scales + fp16 offsets + X + Y.

    q*N*K/8 + 2*q*N*K/G + 2*N*K/G + 2*M*K + 2*M*N
    """
    return q * N * K // 8 + 2 * q * N * (K // G) + 2 * N * (K // G) + 2 * M * K + 2 * M * N


def config0() -> list[Call]:
    """Single 2-bit GEMV, M=1, N=K=4096, G=128."""
    return [Call("o", 1, 4096, 4096, 2)]


def config1_calls() -> list[Call]:
    """8B decode linears at M=1, q in {2,3,4}."""
    return [Call(name, 1, n, k, q) for q in (2, 3, 4) for name, (n, k) in LLAMA31_8B.items()]


def config2_calls() -> list[Call]:
    """Small-batch sweep on the 8B shapes, q in {2,3}, outlier activations."""
    return [Call(name, m, n, k, q, outliers=True)
            for q in (2, 3) for name, (n, k) in LLAMA31_8B.items() for m in (1, 2, 4, 8, 16, 32)]


def config3_calls() -> list[Call]:
    """70B decode linears at M=1, q in {2,3}."""
    return [Call(name, 1, n, k, q) for q in (2, 3) for name, (n, k) in LLAMA31_70B.items()]


def config4_prefill_calls() -> list[Call]:
    """Prefill-sized GEMM on the 8B shapes, q=2."""
    return [Call(name, m, n, k, 2) for name, (n, k) in LLAMA31_8B.items() for m in (128, 512, 2048)]


def config4_stack_calls(layers: int = 32) -> list[Call]:
    """32-layer 8B linear stack at M=1, q=2: 4 linears per layer in model order."""
    out = []
    for layer in range(layers):
        for name in ("qkv", "o", "gate_up", "down"):
            n, k = LLAMA31_8B[name]
            out.append(Call(f"L{layer}.{name}", 1, n, k, 2))
    return out
