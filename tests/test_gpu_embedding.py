"""GPU parity of the gated adaptive embedding (lookup through E G O) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, empty_dev, host, rel_fro, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


# word clusters shaped like the adaptive embedding of the word-level model: reduced dimensions
# 1024 / 256 / 64 projected to d = 1024 (vocabulary sizes scaled down), plus a ragged case
@pytest.mark.parametrize("n_rows,d_i,d,T", [(2000, 1024, 1024, 3000), (4000, 256, 1024, 2500), (5000, 64, 1024, 1111),
                                            (300, 72, 200, 515)])
def test_gated_embedding_matches_oracle(b, n_rows, d_i, d, T):
    g = np.random.default_rng(n_rows + d_i)
    E = I.round_to_bf16(g.standard_normal((n_rows, d_i)).astype(np.float32))
    Om = I.round_to_bf16((g.standard_normal((d_i, d)) / np.sqrt(d_i)).astype(np.float32))
    dY = I.round_to_bf16(g.standard_normal((T, d)).astype(np.float32))
    # word frequencies are heavily skewed: many repeats of a few rows
    ids = np.minimum((g.pareto(1.2, T) * 3).astype(np.int64), n_rows - 1).astype(np.int32)
    alpha = I.log_alpha(("normal", 0.5, 1.5), d_i, 0, 31)
    z, mask, dzd = O.gate_sample(alpha, *HC, seed=0, offset=0)
    z32, dzd32 = z.astype(np.float32), dzd.astype(np.float32)
    bf = torch.bfloat16
    Ed, Od, dYd = to_dev(E, "bf16"), to_dev(Om, "bf16"), to_dev(dY, "bf16")
    idd = torch.from_numpy(ids).cuda()
    zt, dt = torch.from_numpy(z32).cuda(), torch.from_numpy(dzd32).cuda()
    Y, H = empty_dev(T, d, bf), empty_dev(T, d_i, bf)
    b.gated_embedding_fwd(idd, Ed, Od, zt, Y, H)
    dE = torch.zeros(n_rows, d_i, device="cuda")
    dO = empty_dev(d_i, d, bf)
    dla = torch.full((d_i,), float("nan"), device="cuda")
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_EMBEDDING_BWD, T, 0, 0, d_i, b.BF16))
    ws.fill_(0xFF)
    b.gated_embedding_bwd(dYd, idd, Ed, Od, zt, dt, H, dE, dO, dla, ws)
    assert b.device_status() == b.OK
    _, Hp, Yo = O.gated_embedding_fwd(ids, E, Om, z32)
    G = O.gated_embedding_bwd(dY, ids, E, Om, z32, dzd32)
    assert rel_fro(host(H), Hp) < 4e-3 and rel_fro(host(Y), Yo) < 2e-2
    assert rel_fro(host(dO), G["dO"]) < 2e-2
    assert rel_fro(host(dE), G["dE"]) < 2e-2
    assert rel_fro(host(dla), G["dlog_alpha"]) < 2e-2
    # exact structure: unused words and pruned dimensions get exactly zero
    used = np.zeros(n_rows, bool); used[ids] = True
    assert torch.count_nonzero(dE[torch.from_numpy(~used).cuda()]) == 0
    assert np.all(host(dE)[:, z32 == 0] == 0) and np.all(host(H)[:, z32 == 0] == 0)
    # dlog_alpha is summed in a fixed order: bit-reproducible
    dla2 = torch.empty(d_i, device="cuda")
    b.gated_embedding_bwd(dYd, idd, Ed, Od, zt, dt, H, None, None, dla2, ws)
    assert torch.equal(dla, dla2)


def test_embedding_argument_checks(b):
    E = torch.zeros(10, 16, dtype=torch.float32, device="cuda")
    ids = torch.zeros(4, dtype=torch.int32, device="cuda")
    z = torch.ones(16, device="cuda")
    Y = torch.zeros(4, 8, dtype=torch.float32, device="cuda"); H = torch.zeros(4, 16, dtype=torch.float32, device="cuda")
    with pytest.raises(b.FlopError) as e:
        b.gated_embedding_fwd(ids, E, torch.zeros(16, 8, device="cuda"), z, Y, H)       # fp32 storage is not served
    assert e.value.code == b.ERR_UNSUPPORTED
