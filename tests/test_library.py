"""CPU-side checks of the CUDA library: it builds, loads, exports what the header declares, and its
host-only helpers behave. No GPU work is started here."""
import ctypes
import os
import re

import pytest

from paper_2604_06694_b200 import build as akv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    akv_build.build()
    from paper_2604_06694_b200 import binding
    return binding


def test_exports_every_declared_symbol(B):
    hdr = open(os.path.join(ROOT, "include", "audiokv.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = sorted(set(re.findall(r"\b(audiokv_[a-z_]+)\s*\(", hdr)))
    assert {"audiokv_score", "audiokv_smooth", "audiokv_allocate", "audiokv_select_gather", "audiokv_evict"} <= set(names)
    L = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(L, n), f"{n} declared in audiokv.h but not exported"


def test_params_struct_matches_the_library(B):
    import ctypes
    assert B.lib().audiokv_params_size() == ctypes.sizeof(B.audiokv_params)
    # field offsets follow the C layout rules: the last field ends the struct (up to alignment padding)
    last = B.audiokv_params.page_table_stride
    assert last.offset + last.size == ctypes.sizeof(B.audiokv_params)


def test_budget_from_ratio(B):
    assert B.audiokv_budget_from_ratio(0.4, 112, 8192, 32) == int(0.4 * 112 * 8192)
    assert B.audiokv_budget_from_ratio(0.0, 10, 100, 8) == 80          # never below the windows
    assert B.audiokv_budget_from_ratio(1.0, 10, 100, 8) == 1000
    assert B.audiokv_budget_from_ratio(1.5, 10, 100, 8) == -1
    assert B.audiokv_budget_from_ratio(0.5, 0, 100, 8) == -1


def _prob(B, **kw):
    base = dict(dtype=B.AUDIOKV_BF16, n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, seq_lens=[1000, 333],
                window=32, q_strides=(2 * 32 * 8 * 128, 32 * 8 * 128, 8 * 128, 128),
                kv_strides=(2 * 1333 * 128, 128, 1333 * 128), kv_req_offset=[0, 1000 * 128])
    base.update(kw)
    return B.Problem(**base)


def test_sizes_and_param_checks(B):
    p = _prob(B)
    assert B.audiokv_scores_len(p) == 2 * 2 * (968 + 301)
    assert B.audiokv_workspace_bytes(p) > 0
    assert B.audiokv_workspace_bytes_host(p, 10, 10, [400, 200]) > B.audiokv_workspace_bytes(p)
    assert B.audiokv_scores_len(_prob(B, seq_lens=[1000, 32])) == B.AUDIOKV_EINVAL          # L <= W
    assert B.audiokv_scores_len(_prob(B, head_dim=96)) == B.AUDIOKV_EUNSUPPORTED
    assert B.audiokv_scores_len(_prob(B, n_q_heads=7)) == B.AUDIOKV_EINVAL
    assert B.audiokv_scores_len(_prob(B, rho=0.0)) == B.AUDIOKV_EINVAL
    assert B.audiokv_scores_len(_prob(B, alpha=1.5)) == B.AUDIOKV_EINVAL
    assert B.audiokv_scores_len(_prob(B, kv_strides=(2 * 1333 * 128, 132, 1333 * 128))) == B.AUDIOKV_EALIGN
    assert B.audiokv_workspace_bytes(_prob(B, window=0)) == 0
    assert B.audiokv_strerror(B.AUDIOKV_EWORKSPACE) == "workspace too small"


def test_many_requests_and_query_offsets(B):
    """Batches beyond the 64 requests one launch carries are planned (no GPU work here), and a misaligned or
    negative per-request query offset is refused."""
    n = 300
    lens = [200 + 7 * i for i in range(n)]
    cu = [0]
    for L in lens:
        cu.append(cu[-1] + L)
    p = _prob(B, seq_lens=lens, kv_strides=(2 * cu[-1] * 128, 128, cu[-1] * 128),
              kv_req_offset=[c * 128 for c in cu[:-1]])
    assert B.audiokv_scores_len(p) == 4 * sum(L - 32 for L in lens)
    assert B.audiokv_workspace_bytes(p) > 0
    ok = _prob(B, q_req_offset=[64, 0])
    assert B.audiokv_workspace_bytes(ok) > 0
    assert B.audiokv_scores_len(_prob(B, q_req_offset=[4, 0])) == B.AUDIOKV_EALIGN
    assert B.audiokv_scores_len(_prob(B, q_req_offset=[0, -8])) == B.AUDIOKV_EINVAL


def test_reevict_workspace_and_checks(B):
    p = _prob(B)                               # 2 requests x 2 layers x 2 KV heads = 8 heads
    cu = [0, 300, 700, 1000, 1500, 1900, 2000, 2600, 3000]
    assert B.audiokv_reevict_workspace_bytes(p, cu) > 0
    assert B.audiokv_reevict_workspace_bytes(p, [1] + cu[1:]) == 0          # must start at 0
    assert B.audiokv_reevict_workspace_bytes(p, cu[:5] + [1510] + cu[6:]) == 0   # a head no longer than the window


def test_binding_refuses_cpu_tensors(B):
    import torch
    with pytest.raises(ValueError):
        B._dev(torch.zeros(4), "x")
