"""Seeded random shapes through the whole forward pass (prefill and decode) against the oracle.

The fixed cases elsewhere pin the sizes the kernels' bands and tiles switch on; this sweep draws the rest of
the parameter space (group sizes, head_dim, chunk sizes, exponents, window lengths, ragged lengths, dtypes) from
a seeded generator, so that a change which breaks an unlisted combination still fails a test."""
import numpy as np
import pytest

from tests import test_gpu_parity as P

pytestmark = pytest.mark.gpu


def _run(kind, kw, lens, rows, local_blocks):
    try:
        if kind == "prefill":
            P._fwd_prefill_case(P._wl(**kw), rows, local_blocks=local_blocks, min_clean=0.5)
        else:
            P._decode_case(P._wl(kind="decode", **kw), lens, local_blocks=local_blocks)
    except AssertionError as e:
        # a draw whose only (batch, KV head) groups hold a chunk inside the borderline band has nothing left to
        # compare (the harness excludes such rows by design); every other assertion carries a message
        if "too few clean" in str(e):
            return False
        raise AssertionError(f"{kind} {kw} local_blocks={local_blocks}: {e}") from e
    return True


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_any_path(seed):
    rng = np.random.default_rng(seed)
    done = 0
    for _ in range(150):
        g_q = int(rng.choice([1, 2, 4, 8, 16])); h_kv = int(rng.choice([1, 2, 3]))
        blk = int(rng.choice([16, 32, 64, 128]))
        seq = int(rng.integers(1, 40 * blk if blk <= 32 else 2600))
        batch = int(rng.choice([1, 2]))
        kw = dict(seq=seq, h_q=g_q * h_kv, h_kv=h_kv, head_dim=int(rng.choice([64, 128])), block=blk,
                  dtype=str(rng.choice(["bf16", "bf16", "f32"])), alpha=float(rng.choice([1.25, 1.5, 1.5, 2.0, 1.75])),
                  gamma=float(rng.choice([1.0, 2.0, 4.0])), batch=batch, seed=int(rng.integers(0, 1000)),
                  sigma=float(rng.choice([1.0, 10.0, 1e8])))
        L = int(rng.choice([0, 0, 1, 2, 5]))
        kind = str(rng.choice(["prefill", "prefill", "decode"]))
        rows = sorted(set(rng.integers(0, seq, min(seq, 40)).tolist()) | {0, seq - 1})
        lens = [int(rng.integers(1, seq + 1)) for _ in range(batch)]
        done += _run(kind, kw, lens, rows, L)
    print(f"random shapes (any path) seed {seed}: {done} of 150 draws compared, {150 - done} had too few rows or groups "
          "free of borderline chunks")
    assert done >= 140


@pytest.mark.parametrize("seed", [21])
def test_random_shapes_tensor_core_paths(seed):
    """bf16, g_q >= 2, every chunk size and both head dims: mostly shapes the TMA / tcgen05 kernels serve."""
    rng = np.random.default_rng(seed)
    done, swallowed = 0, []
    for _ in range(120):
        g_q = int(rng.choice([2, 4, 8, 16])); h_kv = int(rng.choice([1, 2]))
        seq = int(rng.integers(1, 9000))
        batch = int(rng.choice([1, 2]))
        kw = dict(seq=seq, h_q=g_q * h_kv, h_kv=h_kv, head_dim=int(rng.choice([128, 128, 64])),
                  block=int(rng.choice([16, 32, 64, 128])), dtype="bf16",
                  alpha=float(rng.choice([1.25, 1.5, 1.5, 2.0, 1.6])), gamma=float(rng.choice([1.0, 2.0])), batch=batch,
                  seed=int(rng.integers(0, 1000)), sigma=float(rng.choice([1.0, 10.0, 1e8])),
                  n_planted=int(rng.choice([2, 5, 9])))
        L = int(rng.choice([0, 0, 1, 2, 7]))
        kind = str(rng.choice(["prefill", "prefill", "decode"]))
        rows = sorted(set(rng.integers(0, seq, min(seq, 30)).tolist()) | {0, seq - 1})
        lens = [int(rng.integers(1, seq + 1)) for _ in range(batch)]
        ok = _run(kind, kw, lens, rows, L)
        done += ok
        if not ok:
            swallowed.append((kind, kw, L))
    print(f"random shapes (tensor-core paths) seed {seed}: {done} of 120 draws compared; not compared: {swallowed}")
    # a tensor-core-path draw that cannot be compared is a gap in the sweep, not noise: none is accepted
    assert not swallowed, swallowed
