"""Pins for oracle.storage and for the packed size: the paper's printed BPW and model sizes."""

import os

import pytest

from oracle import layout, storage

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "storage_tables.txt")

MODELS = {
    # blocks, hidden, kv_dim (k and v projections), ffn, vocab
    "llama31_8b": dict(blocks=32, hidden=4096, kv_dim=1024, ffn=14336, vocab=128256),
    "llama31_70b": dict(blocks=80, hidden=8192, kv_dim=1024, ffn=28672, vocab=128256),
}


def _rows():
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            kind, model, q, G, uni, hl = line.split()
            yield kind, model, int(q), int(G), uni, hl


def _trunc2(x):
    return int(x * 100 + 1e-9) / 100.0


def test_bits_per_weight_match_the_paper():
    for kind, _, q, G, uni, hl in _rows():
        if kind != "bpw":
            continue
        assert _trunc2(storage.hlq_bits_per_weight(q, G)) == pytest.approx(float(hl), abs=1e-9)
        if uni != "-":
            assert storage.uniform_bits_per_weight(q, G) == pytest.approx(float(uni), abs=1e-9)


def test_model_sizes_match_the_paper():
    for kind, model, q, G, uni, hl in _rows():
        if kind != "size":
            continue
        m = MODELS[model]
        digits = len(hl.split(".")[1])
        tol = 0.5 * 10 ** (-digits) + 1e-9
        assert storage.llama_model_gib(storage.hlq_bits_per_weight(q, G), **m) == pytest.approx(float(hl), abs=tol)
        assert storage.llama_model_gib(storage.uniform_bits_per_weight(q, G), **m) == pytest.approx(float(uni), abs=tol)


def test_block_weight_count_is_the_218m_of_the_parameter_table():
    m = MODELS["llama31_8b"]
    assert storage.llama_block_weights(m["hidden"], m["kv_dim"], m["ffn"]) == 218_103_808


@pytest.mark.parametrize("q,G,N,K", [(2, 128, 4096, 4096), (3, 128, 28672, 4096), (2, 64, 4096, 14336), (4, 128, 6144, 4096)])
def test_layer_and_packed_bytes_equal_bits_per_weight(q, G, N, K):
    exact = storage.hlq_layer_bytes(q, G, N, K)
    assert exact * 8 == pytest.approx(storage.hlq_bits_per_weight(q, G) * N * K)
    # the device layout adds only its 128-byte header when N % 16 == 0 and K % 512 == 0
    assert layout.packed_bytes(q, G, N, K) == exact + layout.HEADER_BYTES
