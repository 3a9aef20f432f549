"""A bounded device-side wait that runs out: the tensor-core layer kernel reports LAWCAT_ERR_TIMEOUT through dev_status,
returns, and leaves the device usable (its tensor memory was freed: the next ordinary call is parity-green).

Nothing is made to fault or hang. The test only shortens the bound of the kernel's waits, through the library's test hook,
to a few hundred clock cycles, less than any copy or product takes, so the first wait that is not already satisfied gives
up. The kernel itself is the one every other test runs."""
import pytest

from helpers import check, oracle_params
from oracle import lawcat_oracle as O
from paper_2509_18467_b200 import inputs as I

pytestmark = pytest.mark.gpu

NAMES = ["q", "k", "v", "gate", "w_q", "w_k", "W"]


@pytest.mark.parametrize("T", [40, 700])
def test_wait_that_runs_out_is_reported_and_the_device_stays_usable(T):
    import torch
    from paper_2509_18467_b200 import api
    s = I.LayerShape(1, T, 2, 1, 128, 128, dtype="bf16", config_id=91)
    x = I.make(s, NAMES)
    d = {n: api.to_device(v, s.dtype) for n, v in x.items()}
    p = api.params(s.B, s.T, s.H, s.H_kv, s.d_k, s.d_v)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        api.test_set_wait_limit(300)
        api.trace_begin()
        api.lawcat_layer_fwd(p, *[d[n] for n in NAMES], dev_status=status)
        kernels = api.trace_end()   # (waits for the kernel: it must return by itself)
    finally:
        api.test_set_wait_limit(0)
    assert any(k.startswith("layer_tc") for k in kernels)
    torch.cuda.synchronize()
    assert int(status.item()) == 5, int(status.item())          # LAWCAT_ERR_TIMEOUT
    assert api.status_string(5) == "bounded device wait ran out"
    # the same call with the default bound: no status, parity with the oracle
    status.zero_()
    r = api.lawcat_layer_fwd(p, *[d[n] for n in NAMES], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = O.layer_fwd(oracle_params(s), *[x[n] for n in NAMES])
    check(r["o"], ref["o"], "bf16", "o")
    check(r["S_T"], ref["S_T"], "bf16", "S_T", f32_store=True)
