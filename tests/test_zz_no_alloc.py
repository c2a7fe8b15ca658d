"""The allocation-free scoring entry point against the regular one.

Some users of this library cannot allocate device memory when they need scores -- their process
has given all of the GPU to its own pool, or they sit in a loop where cudaMalloc's device-wide
synchronisation is not acceptable.  For them `citrus_importance_static` keeps its scratch in an
array inside the library image.  This file checks, through the C ABI, that it returns what the
first chunk of `citrus_process_chunk` computes for the same instruction queries and keys and what
the fp64 oracle's Eq. 1 column sums give, twice in a row (the second call reuses the array the
first one left dirty), that the calls leave the amount of free device memory unchanged, and that
oversized requests are refused.  It is named to be collected last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle

from paper_2406_12018_b200 import binding, workloads as wl
from paper_2406_12018_b200.binding import Citrus

pytestmark = pytest.mark.gpu
TOL = {"bf16": 2e-2, "fp32": 1e-4}          # same absolute tolerances as the parity tests (normalised scores)


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("fp32", 64)])
def test_static_scores_match_regular_entry_point_twice(dtype, D):
    for call, (L, n_instr, seed) in enumerate([(300, 37, 21), (512, 64, 22)]):
        w = wl.scaled(wl.CONFIGS["mistral7b_layer"], seed=seed, q_heads=8, kv_heads=2, head_dim=D, budget_k=64,
                      chunk_s=512, doc_tokens=L, n_instr=n_instr, dtype=dtype, n_planted=4)
        doc = wl.make_document(w)
        Q, K, V, Qi = doc.Q.cuda(), doc.K.cuda(), doc.V.cuda(), doc.Q_instr.cuda()
        ctx = Citrus(1, w.q_heads, w.kv_heads, D, w.budget_k, w.chunk_s, dtype=dtype)
        ctx.process_chunk(0, Q, K, V, Qi)
        torch.cuda.synchronize()
        want = ctx.step_view(0)[0].clone()                      # [H_kv, L] scores of the existing entry point
        got = torch.full((w.kv_heads, L + 5), -1.0, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if call == 0:
            binding.importance_static(Qi, K, got, status=status)   # the first call on a device does the one-time set-up
            got.fill_(-1.0)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]             # cudaMemGetInfo: the driver's view, not torch's cache
        binding.importance_static(Qi, K, got, status=status)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free entry point changed free device memory"
        assert int(status.item()) == 0                          # no bounded wait expired
        norm = n_instr * (w.q_heads // w.kv_heads)
        err = float((got[:, :L] - want).abs().max()) / norm
        assert err <= TOL[dtype], f"call {call}: normalised score error {err}"
        # against the definition (Eq. 1, s = I, over exactly these keys; no retained cache)
        S = oracle.importance_sum(wl.to_f64(doc.Q_instr), np.zeros((w.kv_heads, 0, D)), wl.to_f64(doc.K))
        err_o = float(np.abs(got[:, :L].double().cpu().numpy() - S).max()) / norm
        assert err_o <= TOL[dtype], f"call {call}: normalised score error against the oracle {err_o}"
        assert np.allclose(got[:, :L].double().cpu().numpy().sum(axis=1), norm, rtol=2e-3)
        assert bool((got[:, L:] == -1.0).all())                 # nothing written past n_keys
        ctx.close()


def test_static_entry_point_rejects_oversized_and_bad_arguments():
    lib = binding.load()
    f = lib.citrus_importance_static
    q = torch.zeros(8, 32, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(16, 8, 128, dtype=torch.bfloat16, device="cuda")
    s = torch.zeros(8, 16, device="cuda")
    args = lambda n_s, n_keys, hq=32: (q.data_ptr(), n_s, k.data_ptr(), n_keys, hq, 8, 128, 0, s.data_ptr(), 16, None, None)
    assert f(*args(4097, 16)) == -2                               # more scoring rows than CITRUS_MAX_INSTR
    assert f(*args(2052, 16)) == -2                               # 32 heads x 2052 rows > 65536 floats of scratch
    assert f(*args(8, 50000)) == -1                               # score_stride < n_keys
    assert f(None, 8, k.data_ptr(), 16, 32, 8, 128, 0, s.data_ptr(), 16, None, None) == -1
    assert f(q.data_ptr(), 8, k.data_ptr(), 16, 32, 8, 64, 0, s.data_ptr(), 16, None, None) == -9   # bf16 needs D = 128
    assert "size" in binding.strerror(-2)
