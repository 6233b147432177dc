"""The no-allocation scoring entry point agrees with the allocating one.

For callers that cannot allocate on the device (a latency-bound frame loop, a
process whose memory belongs to its own pool), xsv_importance_scores_static
keeps its scratch in a fixed array inside the library.  This file is collected
last on purpose: a run that stops at the first failure has then already run
every other test.  It must pass alone in a fresh process and after the others.
"""
import numpy as np
import pytest
import torch

from paper_2602_21780_b200 import binding, synth

pytestmark = pytest.mark.gpu

TOL = 1e-3          # the score tolerance of the parity tests, relative to max|S|


def _inputs(H, F, n_keys, dtype, layer):
    st = synth.Stream(H=H, d=64, F=F, dtype=dtype, layer=layer)
    q, k, _ = st.frame(0)
    keys = np.concatenate([st.frame(t)[1] for t in range(-(-n_keys // F))], axis=1)[:, :n_keys]
    td = torch.float16 if dtype == "fp16" else torch.bfloat16
    return (torch.from_numpy(q).to("cuda:0", td).contiguous(),
            torch.from_numpy(np.ascontiguousarray(keys)).to("cuda:0", td).contiguous())


def _host(x):
    return x.float().cpu().numpy().astype(np.float64)


def test_static_scratch_entry_point_matches_allocating_one_twice():
    # two calls in a row, the second with fewer heads and other data, so that anything the
    # first call left in the shared array would show up if it were read
    from oracle import xsv_oracle as orc
    for H, F, n_keys, dtype, layer in ((16, 1374, 4000, "bf16", 11), (4, 261, 777, "fp16", 12)):
        Q, keys = _inputs(H, F, n_keys, dtype, layer)
        want = binding.importance_scores(Q, keys)
        got = torch.full((n_keys,), float("nan"), device="cuda:0", dtype=torch.float32)
        torch.cuda.synchronize()                                     # the allocating call has returned its scratch
        free_before = torch.cuda.mem_get_info()[0]
        rc = binding.importance_scores_static(Q, keys, got)
        torch.cuda.synchronize()
        assert rc == 0
        assert torch.cuda.mem_get_info()[0] == free_before          # nothing was allocated
        w, g = want.cpu().numpy(), got.cpu().numpy()
        assert np.all(np.isfinite(g))
        assert np.max(np.abs(g - w)) <= TOL * np.max(np.abs(w))
        # and against the definition itself (Eq. 3-7), not only against the other entry point
        ref = orc.importance_scores(_host(Q), _host(keys), 5, 16)
        assert np.max(np.abs(g - ref)) <= TOL * np.max(np.abs(ref))


def test_static_scratch_entry_point_allocates_nothing_once_set_up():
    # the first call on a device for an input type is set-up (the symbol's address is looked up and, with lazy
    # loading, the module is loaded); from the second call on the free memory must not move, with no allocating
    # call in between
    Q, keys = _inputs(8, 300, 1500, "bf16", 13)
    got = torch.empty(1500, device="cuda:0", dtype=torch.float32)
    assert binding.importance_scores_static(Q, keys, got) == 0      # set-up call
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    assert binding.importance_scores_static(Q, keys, got) == 0
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before


def test_static_scratch_entry_point_rejects_sizes_beyond_its_limit():
    Q = torch.zeros(65, 8, 64, device="cuda:0", dtype=torch.float16)
    keys = torch.zeros(65, 16, 64, device="cuda:0", dtype=torch.float16)
    out = torch.zeros(16, device="cuda:0", dtype=torch.float32)
    rc = binding.importance_scores_static(Q, keys, out)
    assert rc == 9
    assert b"no-allocation" in binding.load().xsv_strerror(rc)
