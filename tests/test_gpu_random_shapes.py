"""GPU parity on seeded random shapes: the two-stage call (pyramidsd_verify_ex) on batches, window lengths and
vocabulary sizes drawn at random -- odd sizes that take the three-pass kernel, sizes of a few tiles with a ragged tail
that take the cluster kernels -- with a random pairing of acceptance modes (Sec. 3.1, 3.2, 3.4), a random schedule
and thresholds placed inside the spread of each stage's divergences, each case against the oracle element by element."""
import numpy as np
import pytest
import torch

from parity_utils import gpu_stage_to_numpy, host_bits
from test_gpu_pyramid_ex import check_pyramid_ex

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def psd():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_12966_b200 import binding
    binding.load_library()
    torch.cuda.set_device(0)
    return binding


@pytest.fixture(scope="module")
def wl():
    from paper_2510_12966_b200 import workloads
    return workloads


def draw_case(case):
    """Shape, dtype, modes and schedule of one case; everything follows from the case number."""
    r = np.random.default_rng(1000 + case)
    dtype = ("f32", "bf16")[case % 2]
    family = case % 4
    if family == 0:      # odd and tiny: the three-pass kernel
        V = int(r.integers(3, 3000)) | 1
    elif family == 1:    # a multiple of the vector width just above the cluster kernel's minimum
        V = 2048 + 8 * int(r.integers(0, 1500))
    elif family == 2:    # several chunks per slice and a ragged tail
        V = 8 * int(r.integers(4000, 9000))
    else:                # even but not a multiple of the vector width
        V = 2 * int(r.integers(2000, 20000)) + 2
    K_d = int(r.integers(1, 13))
    K_q = int(r.integers(1, K_d + 1))
    B = int(r.integers(1, 25))
    modes = [int(m) for m in r.integers(0, 4, size=2)]
    schedule = int(r.integers(0, 5))
    return dict(dtype=dtype, V=V, K_d=K_d, K_q=K_q, B=B, modes=modes, schedule=schedule,
                seed=int(r.integers(0, 2**31)), offset=int(r.integers(0, 1000)))


@pytest.mark.parametrize("case", range(24))
def test_random_shape_against_oracle(psd, oracle, wl, case):
    c = draw_case(case)
    mode_of = {0: psd.FUZZY, 1: psd.STRICT, 2: psd.FUZZY_SD_FALLBACK, 3: psd.ASSISTED}
    mode_q, mode_t = mode_of[c["modes"][0]], mode_of[c["modes"][1]]
    dev = torch.device("cuda:0")
    zd, zq, zt, tok = wl.make_pyramid_inputs(c["B"], c["K_d"], c["K_q"], c["V"], c["dtype"], seed=300 + case,
                                             sigma_q=0.3, sigma_d=0.6)
    hosts = tuple(host_bits(t) for t in (zd, zq, zt))
    dd = [t.to(dev) for t in (zd, zq, zt, tok)]
    # thresholds at the median of each stage's divergences, a probe call's, moved off every value by half the gap to
    # its neighbour: some rows pass, some fail, none sits on the threshold
    probe = psd.verify_ex(*dd, 1e9, 1e9, psd.FUZZY, psd.FUZZY, 1, 1)
    torch.cuda.synchronize()

    def between(values):
        v = np.unique(values[np.isfinite(values)])
        if len(v) < 2:
            return float(v[0]) + 1.0 if len(v) else 0.5
        i = len(v) // 2
        return float(0.5 * (v[i - 1] + v[i]))

    tau_q = between(probe["div_q"].cpu().numpy().ravel())
    tau_t = between(probe["div_t"].cpu().numpy().ravel())
    out = psd.verify_ex(*dd, tau_q, tau_t, mode_q, mode_t, c["seed"], c["offset"], schedule=c["schedule"])
    torch.cuda.synchronize()
    assert psd.last_status() == 0
    gpu = gpu_stage_to_numpy(out)
    ties, n, orc = check_pyramid_ex(oracle, gpu, hosts, tok.numpy(), c["dtype"], mode_q, mode_t, tau_q, tau_t,
                                    c["seed"], c["offset"])
    assert ties <= 2 and n >= c["B"] - 2
    assert orc["accept_len_q"].min() >= 0 and orc["accept_len"].max() <= c["K_q"]
