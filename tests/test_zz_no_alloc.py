"""``fastav_select_noalloc``: the selection step for callers that cannot allocate device memory.

Some users of the library prune from a place where no device allocation is possible: a plug-in that
is handed input and output tensors only, a latency-critical loop that must not hit cudaMalloc's
implicit synchronisation, a process whose memory pool was fully assigned at start-up.  For them the
library carries its own scratch (a fixed array of keys, one per token, 4 MiB) and this entry point
uses it instead of a workspace.  The test calls it through the C ABI twice in a row on different
inputs -- the second call finds the first call's keys still in the array -- and requires the same
keep lists as ``fastav_select`` gives, and as the CPU oracle's selector gives on the same scores, bit
for bit (integer work: no tolerance).  The file sorts last so that a run stopping at the first failure
has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2601_13143_b200 import fastav

pytestmark = pytest.mark.gpu


def _problem(seed, lens, keeps, rows):
    rng = np.random.default_rng(seed)
    n = sum(lens)
    scores = (rng.integers(0, 4000, size=n) / 65536.0).astype(np.float32)     # many exact ties
    protect = (rng.random(n) < 0.02).astype(np.uint8)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    cuq = np.concatenate([[0], np.cumsum(rows)]).astype(np.int32)
    q_idx = np.concatenate([np.arange(n_b - r, n_b) for n_b, r in zip(lens, rows)]).astype(np.int32)
    params = fastav.make_params(batch=len(lens), total_tokens=n, max_seqlen=max(lens), total_q=int(cuq[-1]), max_qlen=max(rows),
                                total_keep=sum(keeps), max_keep=max(keeps), num_q_heads=4, num_kv_heads=2, head_dim=64,
                                hidden=64, flags=fastav.FASTAV_PROTECT_QUERY_ROWS)
    dev = lambda a, dt: torch.as_tensor(a, dtype=dt).cuda()
    host = dict(scores=scores, cu=cu, keeps=np.asarray(keeps, dtype=np.int32), protect=protect, q_idx=q_idx, cuq=cuq)
    return dict(host=host, params=params, scores=dev(scores, torch.float32), cu=dev(cu, torch.int32), keeps=dev(keeps, torch.int32),
                protect=dev(protect, torch.uint8), q_idx=dev(q_idx, torch.int32), cuq=dev(cuq, torch.int32),
                total_keep=sum(keeps), batch=len(lens))


def _outputs(pr):
    return (torch.full((pr["total_keep"] + 8,), -7, dtype=torch.int32, device="cuda"),
            torch.full((pr["batch"] + 1,), -7, dtype=torch.int32, device="cuda"),
            torch.zeros(1, dtype=torch.int32, device="cuda"))


def test_select_noalloc_matches_select_on_two_calls_in_a_row():
    # the first problem has a sequence longer than fits in shared memory, the second is short and ragged
    problems = [_problem(11, [70_000, 513, 0, 4096], [23_000, 100, 0, 4096], [4, 1, 0, 2]),
                _problem(12, [1000, 7, 129], [400, 7, 1], [1, 1, 3])]
    for pr in problems:
        ws = torch.empty(max(fastav.fastav_workspace_bytes(pr["params"]), 256), dtype=torch.uint8, device="cuda")
        want_idx, want_cu, want_status = _outputs(pr)
        fastav.fastav_select(pr["params"], pr["scores"], pr["cu"], pr["keeps"], pr["protect"], pr["q_idx"], pr["cuq"],
                             want_idx, want_cu, ws, want_status)
        got_idx, got_cu, got_status = _outputs(pr)
        fastav.fastav_select_noalloc(pr["params"], pr["scores"], pr["cu"], pr["keeps"], pr["protect"], pr["q_idx"], pr["cuq"],
                                     got_idx, got_cu, got_status)
        torch.cuda.synchronize()
        assert torch.equal(got_cu, want_cu)
        assert int(want_cu[-1]) == pr["total_keep"]
        assert torch.equal(got_idx, want_idx)                  # includes the untouched guard entries past the end
        assert int(got_status) == int(want_status)
        # ... and both are what the plain definition gives (score descending, index ascending, protected first)
        h = pr["host"]
        ref_idx, ref_cu = oracle.select(h["scores"], h["cu"], h["keeps"], h["protect"], True, h["q_idx"], h["cuq"])
        assert got_cu.cpu().tolist() == ref_cu.tolist()
        assert np.array_equal(got_idx.cpu().numpy()[:pr["total_keep"]], ref_idx)


def test_select_noalloc_rejects_sizes_beyond_its_scratch():
    too_many = fastav.NOALLOC_MAX_TOKENS + 1
    params = fastav.make_params(batch=1, total_tokens=too_many, max_seqlen=too_many, total_q=0, max_qlen=0, total_keep=1,
                                max_keep=1, num_q_heads=4, num_kv_heads=2, head_dim=64, hidden=64)
    fake = ctypes.c_void_p(0x1000)   # never dereferenced: the size check comes first and nothing is launched
    rc = fastav.library().fastav_select_noalloc(ctypes.byref(params), fake, fake, fake, None, None, None, fake, fake, None, None)
    assert rc == fastav.FASTAV_ERR_UNSUPPORTED
