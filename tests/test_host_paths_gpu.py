"""GPU tests of the boundary's host-side rules: the time-out report, stream ordering of a position-shift context,
and the two input-ordering routes."""
import pytest
import torch

from paper_2406_12018_b200 import workloads as wl
from paper_2406_12018_b200.binding import Citrus
import parity_util as pu

pytestmark = pytest.mark.gpu
C = wl.CONFIGS


def test_an_expired_device_wait_is_reported_once_and_the_context_stays_usable():
    # Every wait inside the kernels is bounded; one that runs out raises the context's status word and the kernel
    # returns.  Here a one-warp kernel waits one millisecond on an mbarrier that nothing arms (no fault, no trap, no
    # endless loop), with the same wait routine the product kernels use.
    w = wl.scaled(C["mistral7b_layer"], q_heads=8, kv_heads=2, budget_k=256, chunk_s=256, doc_tokens=600, n_instr=24,
                  n_planted=4)
    ctx = pu.make_pair(w)
    assert ctx.poll_status() == 0
    ctx.debug_expire_wait(1_000_000)
    assert ctx.poll_status() == -8                         # CITRUS_ERR_TIMEOUT
    assert ctx.poll_status() == 0                          # the read cleared the word
    # the CUDA context is intact: a document still goes through with parity
    _, st = pu.run_document(w, ctx)
    assert st["checked_chunks"] == 3 and ctx.poll_status() == 0
    ctx.close()


def test_position_shift_slots_stepped_on_two_streams_do_not_share_scratch_in_time():
    # a position-shift context embeds every step into one scratch: steps of two slots submitted on two streams must
    # still give what the same steps give one after the other on one stream
    w = wl.scaled(C["tiny_fp32"], q_heads=8, kv_heads=2, head_dim=128, budget_k=200, chunk_s=160, doc_tokens=960,
                  n_instr=12, dtype="bf16", mode="shared", n_planted=4, n_sinks=1, position_shift=True, n_seqs=2)
    docs = [wl.make_document(w, seq=s) for s in range(2)]
    dev = [[t.cuda() for t in (d.Q, d.K, d.V, d.Q_instr)] for d in docs]
    a, b = pu.make_pair(w), pu.make_pair(w)
    s0, s1 = torch.cuda.Stream(), torch.cuda.Stream()
    outs_a = [torch.empty_like(dev[s][0]) for s in range(2)]
    outs_b = [torch.empty_like(dev[s][0]) for s in range(2)]
    torch.cuda.synchronize()
    for c in range(0, 960, 160):
        sl = slice(c, c + 160)
        for s, st in ((0, s0), (1, s1)):
            Q, K, V, Qi = dev[s]
            a.process_chunk(0, Q[sl], K[sl], V[sl], Qi, out=outs_a[s][sl], slot=s, stream=st)
    torch.cuda.synchronize()
    for c in range(0, 960, 160):
        sl = slice(c, c + 160)
        for s in range(2):
            Q, K, V, Qi = dev[s]
            b.process_chunk(0, Q[sl], K[sl], V[sl], Qi, out=outs_b[s][sl], slot=s)
            torch.cuda.synchronize()
    for s in range(2):
        assert torch.equal(outs_a[s], outs_b[s])
        for x, y in zip(a.cache_view(0, 0, s), b.cache_view(0, 0, s)):
            assert torch.equal(x, y)
    assert a.poll_status() == 0
    a.close(); b.close()


@pytest.mark.parametrize("mode", ["shared", "individual"])
def test_inputs_ready_route_equals_the_default_route(mode):
    # default: every kernel of a call waits for earlier stream work before its first load of the caller's tensors;
    # with the caller's promise that inputs are complete the chunk's tiles are loaded early.  Same results, bit for bit,
    # also when the calls are enqueued back to back without synchronisation.
    w = wl.scaled(C["mistral7b_layer"], budget_k=384, chunk_s=256, doc_tokens=2048 + 100, n_instr=40, mode=mode,
                  lm_window=48, n_planted=6)
    doc = wl.make_document(w)
    Q, K, V, Qi = (t.cuda() for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
    res = []
    for ready in (False, True):
        ctx = pu.make_pair(w)
        ctx.set_inputs_ready(ready)
        out = torch.empty_like(Q)
        torch.cuda.synchronize()
        for c in range(0, Q.shape[0], w.chunk_s):
            sl = slice(c, min(Q.shape[0], c + w.chunk_s))
            ctx.process_chunk(0, Q[sl], K[sl], V[sl], Qi, out=out[sl])
        torch.cuda.synchronize()
        views = [tuple(t.clone() for t in ctx.cache_view(0, cid)) for cid in range(2 if mode == "individual" else 1)]
        res.append((out, views))
        assert ctx.poll_status() == 0
        ctx.close()
    assert torch.equal(res[0][0], res[1][0])
    for va, vb in zip(res[0][1], res[1][1]):
        for x, y in zip(va, vb):
            assert torch.equal(x, y)
    # and the fast route against the oracle, whole document
    ctx = pu.make_pair(w)
    ctx.set_inputs_ready(True)
    _, st = pu.run_document(w, ctx)
    assert st["checked_chunks"] == 9
    ctx.close()


def test_attention_beside_the_scoring_chain_gives_the_same_bits_as_one_stream():
    # Shared cache scored by the instruction text: nothing in a2-a4 reads a1's result, and a step of at most 64 attention
    # items (here 2 row tiles x 32 heads) runs a1 on a side stream beside log-sum-exp -> column sums -> select / gather.
    # Off (0), the default and a larger limit must agree bit for bit, with the calls enqueued back to back; the
    # caller's stream alone orders `out` and the caches.
    w = wl.scaled(C["mistral7b_layer"], chunk_s=256, doc_tokens=4096 + 100, n_planted=6)
    doc = wl.make_document(w)
    Q, K, V, Qi = (t.cuda() for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
    res = []
    for cap in (0, None, 148):
        ctx = pu.make_pair(w)
        ctx.set_inputs_ready(True)
        if cap is not None:
            ctx.set_attention_beside(cap)
        out = torch.empty_like(Q)
        st = torch.cuda.Stream()
        torch.cuda.synchronize()
        with torch.cuda.stream(st):
            for c in range(0, Q.shape[0], w.chunk_s):
                sl = slice(c, min(Q.shape[0], c + w.chunk_s))
                ctx.process_chunk(0, Q[sl], K[sl], V[sl], Qi, out=out[sl], stream=st)
            seen = out.float().abs().sum()                 # stream-ordered read of `out` right behind the last call
        torch.cuda.synchronize()
        assert float(seen) == float(out.float().abs().sum())
        res.append((out, tuple(t.clone() for t in ctx.cache_view(0, 0))))
        assert ctx.poll_status() == 0
        ctx.close()
    for out, view in res[1:]:
        assert torch.equal(res[0][0], out)
        for x, y in zip(res[0][1], view):
            assert torch.equal(x, y)
    # and through a CUDA graph: the side stream joins the capture and leaves it again inside every call
    ctx = pu.make_pair(w)
    ctx.set_inputs_ready(True)
    out = torch.empty_like(Q)
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(g, stream=st):
        for c in range(0, Q.shape[0], w.chunk_s):
            sl = slice(c, min(Q.shape[0], c + w.chunk_s))
            ctx.process_chunk(0, Q[sl], K[sl], V[sl], Qi, out=out[sl], stream=st)
    ctx.reset()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(res[0][0], out) and ctx.poll_status() == 0
    ctx.close()
