"""The scratch-free variant of tile construction, for callers that cannot allocate device memory
(serving loops that must not touch the allocator, plug-ins that only receive their buffers, memory
managers that forbid allocation after start-up).  It must give what the ordinary entry point gives:
identical tile bits, alpha within the tolerance the other tests use -- on two calls in a row, because
every call reuses the same built-in scratch array and has to leave it fit for the next one.
This file sorts last on purpose, so a run that stops at the first failure has run everything else."""
import numpy as np
import pytest
import torch

from oracle import tbn_oracle as O
from paper_2407_12075_b200 import binding as B
from paper_2407_12075_b200 import synth
from tests.util import to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("N,k,mode", [(512 * 512, 4, B.ALPHA_PER_TILE), (2304 * 768, 8, B.ALPHA_PER_LAYER),
                                      (7 * 33, 3, B.ALPHA_PER_TILE)])
def test_static_scratch_entry_point_matches_ordinary_one_twice(N, k, mode):
    results = []
    for call in range(2):                       # second call sees the first call's leftovers in the array
        W_np, A_np = synth.normal(40 + call, 1, N, 0.02), synth.normal(40 + call, 101, N, 0.05)
        W, A = to_dev(W_np), to_dev(A_np)
        tile_ref, alpha_ref = B.tbn_aggregate_tile(W, k, mode, A=A)
        tile = torch.full_like(tile_ref, -1)
        alpha = torch.full_like(alpha_ref, float("nan"))
        B.tbn_aggregate_tile_static(W, k, tile, alpha, mode, A=A)
        torch.cuda.synchronize()
        assert torch.equal(tile, tile_ref), f"call {call}: tile bits differ"
        assert np.allclose(alpha.cpu().numpy(), alpha_ref.cpu().numpy(), rtol=1e-6, atol=0), f"call {call}"
        # and against the CPU definition directly, not only through the other entry point
        words, al = O.prepare(W_np, k, mode == B.ALPHA_PER_TILE, A=A_np)
        assert np.array_equal(tile.cpu().numpy().view(np.uint32), words), f"call {call}: tile bits differ from the oracle"
        assert np.allclose(alpha.cpu().numpy(), al, rtol=1e-6, atol=0), f"call {call}: alpha differs from the oracle"
        results.append(tile.clone())
    assert not torch.equal(results[0], results[1])      # the two calls really had different inputs


def test_static_scratch_limit_is_exact():
    # one-element tiles (q = 1) need 16 + 8 k bytes of scratch: k = 131070 is the largest that fits the 1 MiB array,
    # k = 131071 is refused before anything is launched
    k = 131070
    W_np = synth.normal(44, 1, k, 0.02)
    W = to_dev(W_np)
    tile = torch.full((B.tbn_tile_words(1),), -1, dtype=torch.int32, device=W.device)
    alpha = torch.full((k,), float("nan"), dtype=torch.float32, device=W.device)
    B.tbn_aggregate_tile_static(W, k, tile, alpha, B.ALPHA_PER_TILE)
    torch.cuda.synchronize()
    words, al = O.prepare(W_np, k, True)
    assert np.array_equal(tile.cpu().numpy().view(np.uint32), words)
    assert np.allclose(alpha.cpu().numpy(), al, rtol=1e-6, atol=0)
    W1 = to_dev(synth.normal(44, 1, k + 1, 0.02))
    alpha1 = torch.empty(k + 1, dtype=torch.float32, device=W.device)
    with pytest.raises(B.TbnError) as e:
        B.tbn_aggregate_tile_static(W1, k + 1, tile, alpha1, B.ALPHA_PER_TILE)
    assert e.value.status == -4
