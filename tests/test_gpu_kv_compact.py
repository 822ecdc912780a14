"""GPU parity: jet_kv_compact against the oracle, byte-exact over the whole cache."""
import numpy as np
import pytest

from jet_inputs import make_paged_cache
from oracle import kv_compact_ref

pytestmark = pytest.mark.gpu


def _rand_bits(rng, shape):
    return rng.integers(0, 1 << 16, size=shape).astype(np.uint16)


def _random_paths(rng, batch, B, N, accept):
    path = np.full((batch, N + 1), -1, dtype=np.int32)
    for b in range(batch):
        nodes = np.sort(rng.choice(np.arange(1, B), size=accept[b], replace=False)) if accept[b] else []
        path[b, 0] = 0
        path[b, 1:1 + accept[b]] = nodes
    return path


@pytest.mark.parametrize("layers,batch,B,Hkv,D,N,Lmax", [(1, 1, 16, 2, 64, 4, 530), (36, 1, 64, 8, 128, 8, 140),
                                                          (3, 4, 33, 4, 128, 12, 77), (2, 2, 512, 1, 8, 64, 70)])
def test_contiguous(layers, batch, B, Hkv, D, N, Lmax):
    rng = np.random.default_rng(layers * 100 + batch)
    import jet_harness as H
    tk, tv = _rand_bits(rng, (layers, batch, B, Hkv, D)), _rand_bits(rng, (layers, batch, B, Hkv, D))
    kc, vc = _rand_bits(rng, (layers, batch, Lmax, Hkv, D)), _rand_bits(rng, (layers, batch, Lmax, Hkv, D))
    accept = rng.integers(0, min(N, B - 1) + 1, size=batch)
    accept[0] = min(N, B - 1)
    if batch > 1:
        accept[1] = 0
    seq = rng.integers(0, Lmax - N - 1, size=batch).astype(np.int32)
    path = _random_paths(rng, batch, B, N, accept)
    rk, rv, rs = kv_compact_ref(tk, tv, kc, vc, None, path, accept, seq)
    gk, gv, gs = H.run_kv_compact(tk, tv, kc, vc, None, path, accept, seq, N)
    assert np.array_equal(gs, rs)
    assert np.array_equal(gk, rk) and np.array_equal(gv, rv)
    assert not np.array_equal(gk, kc)


@pytest.mark.parametrize("layers,batch,B,Hkv,D,N", [(2, 3, 16, 2, 64, 4), (36, 4, 64, 8, 128, 8)])
def test_paged_page16_shuffled_table(layers, batch, B, Hkv, D, N):
    rng = np.random.default_rng(layers + batch)
    import jet_harness as H
    seq = rng.integers(1, 200, size=batch).astype(np.int32)
    seq[0] = 15                                     # the commit straddles a page boundary
    k0, v0, table = make_paged_cache(rng, seq, 16, Hkv, D, reserve=N + 1)
    kc = np.stack([_rand_bits(rng, k0.shape) for _ in range(layers)])
    vc = np.stack([_rand_bits(rng, k0.shape) for _ in range(layers)])
    tk, tv = _rand_bits(rng, (layers, batch, B, Hkv, D)), _rand_bits(rng, (layers, batch, B, Hkv, D))
    accept = rng.integers(0, N + 1, size=batch)
    accept[0] = N
    path = _random_paths(rng, batch, B, N, accept)
    rk, rv, rs = kv_compact_ref(tk, tv, kc, vc, table, path, accept, seq)
    gk, gv, gs = H.run_kv_compact(tk, tv, kc, vc, table, path, accept, seq, N)
    assert np.array_equal(gs, rs)
    assert np.array_equal(gk, rk) and np.array_equal(gv, rv)
