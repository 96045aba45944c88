"""c2r_permute_static: the dispatch for callers that cannot provide (or allocate) device scratch.

Some users of this library sit where no device memory can be obtained at call time: the process
has given all of it to its own pool, the host application forbids allocation on the request path,
or a cudaMalloc's device-wide synchronisation would break a latency budget.  For them the library
carries its own fixed scratch; this file checks that the variant gives exactly what c2r_permute
gives, twice in a row (the second call sees the first call's leftovers in the shared array), and
that a batch beyond the built-in limit is refused with its own error code.

Collected last on purpose (the file name sorts after every other test file), so a run that stops
at the first failure has already run everything else.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2504_01337_b200 import inputs as G

pytestmark = pytest.mark.gpu


def _outputs(b, cfg, E, K, N, d, dtype):
    R = b.permuted_rows(cfg)
    return dict(counts=torch.full((E,), -3, dtype=torch.int32, device="cuda"),
                offsets=torch.full((E + 1,), -3, dtype=torch.int32, device="cuda"),
                ros=torch.full((N * K,), -3, dtype=torch.int32, device="cuda"),
                sor=torch.full((R,), -3, dtype=torch.int32, device="cuda"),
                Xp=torch.full((R, d), 5.0, dtype=dtype, device="cuda"),
                status=torch.zeros(1, dtype=torch.int32, device="cuda"))


def test_static_scratch_permute_matches_workspace_permute_twice():
    from paper_2504_01337_b200 import binding as b
    cases = [  # two different batches back to back: different sizes, experts, alignment, dtype
        dict(N=16384, K=4, E=60, d=256, align=128, bf16=True, seed=1),
        dict(N=3001, K=2, E=8, d=64, align=1, bf16=False, seed=2),
    ]
    for c in cases:
        N, K, E, d = c["N"], c["K"], c["E"], c["d"]
        cfg = b.make_config(N, d, E, 16, K, K - 1, 1, 0, b.BF16 if c["bf16"] else b.F32, c["align"])
        dtype = torch.bfloat16 if c["bf16"] else torch.float32
        L = G.random_logits(c["seed"], N, E)
        idx = torch.from_numpy(np.argsort(-L, axis=1, kind="stable")[:, :K].astype(np.int32)).cuda()
        rank = torch.from_numpy(np.random.default_rng(c["seed"]).permutation(E).astype(np.int32)).cuda()
        X = torch.from_numpy(G.normal(c["seed"], G.S_X, (N, d))).to(dtype).cuda()
        ref = _outputs(b, cfg, E, K, N, d, dtype)
        ws = torch.empty(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
        b.permute(cfg, idx, rank, X, ref["counts"], ref["offsets"], ref["ros"], ref["sor"], ref["Xp"], ref["status"], ws)
        got = _outputs(b, cfg, E, K, N, d, dtype)
        b.permute_static(cfg, idx, rank, X, got["counts"], got["offsets"], got["ros"], got["sor"], got["Xp"],
                         got["status"])
        torch.cuda.synchronize()
        for name in ref:  # integer index work and row copies: bit-exact
            assert torch.equal(got[name], ref[name]), name
        assert int(got["counts"].sum()) == N * K


@pytest.mark.parametrize("N", [150000, 559232])
def test_static_scratch_large_batches_match_the_oracle(N):
    """Index-only dispatch of batches past 1024 sort blocks (separate histogram / scan / rank launches),
    the second one filling the built-in scratch to its last byte (4369 blocks * 60 experts * 4 B <= 1 MiB),
    through both entry points, against the oracle."""
    from oracle import c2r_oracle as O
    from paper_2504_01337_b200 import binding as b
    E, K, align = 60, 4, 128
    rng = np.random.default_rng(N)
    idx = np.argsort(-rng.standard_normal((N, E)).astype(np.float32), axis=1, kind="stable")[:, :K].astype(np.int32)
    rank = rng.permutation(E).astype(np.int32)
    cfg = b.make_config(N, 64, E, 16, K, K - 1, 1, 0, b.BF16, align)
    assert b.workspace_bytes(cfg, b.WS_PERMUTE) <= (1 << 20)
    ref = O.permute_index(idx, E, rank, align)
    idx_d, rank_d = torch.from_numpy(idx).cuda(), torch.from_numpy(rank).cuda()
    ws = torch.empty(b.workspace_bytes(cfg, b.WS_PERMUTE), dtype=torch.uint8, device="cuda")
    for static in (False, True):
        o = _outputs(b, cfg, E, K, N, 1, torch.bfloat16)
        if static:
            b.permute_static(cfg, idx_d, rank_d, None, o["counts"], o["offsets"], o["ros"], o["sor"], None, o["status"])
        else:
            b.permute(cfg, idx_d, rank_d, None, o["counts"], o["offsets"], o["ros"], o["sor"], None, o["status"], ws)
        torch.cuda.synchronize()
        assert np.array_equal(o["counts"].cpu().numpy(), ref[0]) and np.array_equal(o["offsets"].cpu().numpy(), ref[1])
        assert np.array_equal(o["ros"].cpu().numpy(), ref[2])
        sor = o["sor"].cpu().numpy()
        assert np.array_equal(sor[: ref[3].size], ref[3]) and np.all(sor[ref[3].size:] == -1)
        assert int(o["status"].item()) == 0


def test_static_scratch_limit_is_an_error_code():
    from paper_2504_01337_b200 import binding as b
    # ceil(N/128) * E * 4 bytes = 4688 * 64 * 4 > 1 MiB: refused on the host, nothing is dereferenced
    cfg = b.make_config(600000, 64, 64, 16, 4, 3, 1, 0, b.BF16, 1)
    t = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(b.C2RError) as e:
        b.permute_static(cfg, t, None, None, t, t, t, t, None, None)
    assert e.value.code == -5
    # the workspace variant accepts the same shape when given enough scratch
    assert b.workspace_bytes(cfg, b.WS_PERMUTE) > (1 << 20)
