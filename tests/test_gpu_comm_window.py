"""The real communication window (one-shot all-reduce fused into the window kernel) on ONE GPU.

No second rank runs here: the peers' exchange blocks are blocks of this process on the same GPU,
filled by the test, and the peers' arrival flags are set from the host before the step is queued,
so no kernel ever waits for another launch.  The code path is the multi-GPU one (peer pointers,
system-scope flag protocol, device-side epochs).  Parity bar as in test_gpu_parity.py."""
import numpy as np
import pytest
import torch

from paper_2501_08192_b200 import binding as P
from paper_2501_08192_b200 import inputs as I

import gpu_util as G

pytestmark = pytest.mark.gpu

FAR = 0x3FFFFFFF      # "has announced every window up to this epoch"


def make_ranks(shape, my_rank):
    """One Comm per rank of the shard group, all in this process, mutually connected."""
    comms = [P.Comm(r, shape.tp_degree, shape.batch, shape.hidden) for r in range(shape.tp_degree)]
    for a in comms:
        for b in comms:
            if a is not b:
                a.set_peer(b)
    return comms


def fill_peer_buffers(comms, my_rank, t, own_a_bits):
    """Window A: rank p's buffer = partials_in[p]; window B: peers' buffers = attn_peer_partials."""
    P_ = len(comms)
    for p, c in enumerate(comms):
        c.write(0, G.bits_to_cuda(own_a_bits if p == my_rank else t["partials_in"][p]))
    peers = [p for p in range(P_) if p != my_rank]
    for i, p in enumerate(peers):
        comms[p].write(1, G.bits_to_cuda(t["attn_peer_partials"][i]))
    torch.cuda.synchronize()


@pytest.mark.parametrize("batch,P_,rank,hidden", [(5, 3, 1, 512), (24, 4, 0, 2048), (3, 2, 1, 2048), (8, 8, 7, 1024)],
                         ids=["gemv_p3", "tensor_p4", "cluster_p2", "p8"])
def test_fused_allreduce_window_matches_the_oracle(oracle, batch, P_, rank, hidden):
    shape = I.small_shape(name="comm", batch=batch, hidden=hidden, ffn=256, tp_degree=P_, ctx=140, ctx_min=6, seed=81)
    t = I.make_layers(shape, 1)[0]
    # the oracle sums the same P buffers; in the real window this rank's own window-A contribution is
    # partials_in[rank] (what its previous down projection would have written)
    ref = oracle.layer_step(shape, t)
    comms = make_ranks(shape, rank)
    dl = G.DeviceLayer(shape, t)
    stream = torch.cuda.Stream()
    try:
        fill_peer_buffers(comms, rank, t, t["partials_in"][rank])
        me = comms[rank]
        for p in range(P_):
            if p != rank:
                me.debug_arrive(0, p, FAR)
                me.debug_arrive(1, p, FAR)
        dl.layer.set_comm(me)
        base = None
        for rep in range(3):
            # window A's own buffer is overwritten by the step's down projection: restore it
            me.write(0, G.bits_to_cuda(t["partials_in"][rank]))
            torch.cuda.synchronize()
            with torch.cuda.stream(stream):
                dl.run(stream)
            stream.synchronize()
            assert dl.layer.last_status_code() == 0
            out, inter = dl.outputs(), dl.intermediates()
            for name in ("h", "x", "x2"):
                G.assert_close(inter[name], ref[name], f"{name} (rep {rep})")
            for name in ("attn_partial", "h2", "mlp_partial"):
                G.assert_close(out[name], ref[name], f"{name} (rep {rep})")
            bits = dl.output_bits()
            if base is None:
                base = bits
            for k in base:
                assert np.array_equal(base[k], bits[k]), k
            # device-side epochs: one more completed window of each kind per step, no host involvement
            assert me.epoch(0) == rep + 1 and me.epoch(1) == rep + 1
        # the step announced itself in every peer's flag block (row of window 0 / 1, column = this rank)
        assert dl.layer.graph_captures() == 1
        # the down projection left this rank's MLP partial sums in its window-A buffer for the next step
        dl.layer.set_comm(None)
        dl.run()
        assert dl.layer.last_status() == P.PRESERVE_OK
        G.assert_close(dl.outputs()["mlp_partial"], ref["mlp_partial"], "stand-in again after detaching")
    finally:
        dl.close()
        for c in comms:
            c.close()


def test_a_peer_that_never_arrives_ends_the_wait_with_a_status(oracle):
    """Rank 2 never announces its window-B buffer (a flag that nothing sets): the window kernel's
    wait, limited to about a millisecond for the test, gives up; the step returns; the status names
    the peer wait; with the flag set the same handle works again."""
    shape = I.small_shape(name="comm_timeout", batch=4, hidden=512, ffn=256, tp_degree=3, ctx=50, seed=82)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t)
    rank = 0
    comms = make_ranks(shape, rank)
    dl = G.DeviceLayer(shape, t)
    stream = torch.cuda.Stream()
    try:
        fill_peer_buffers(comms, rank, t, t["partials_in"][rank])
        me = comms[rank]
        me.debug_arrive(0, 1, FAR)
        me.debug_arrive(0, 2, FAR)
        me.debug_arrive(1, 1, FAR)           # rank 2's window-B flag stays at zero
        dl.layer.set_comm(me)
        dl.layer.debug_set(P.DEBUG_WAIT_LIMIT_CYCLES, 1 << 21)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            dl.run(stream)
            e1.record(stream)
        stream.synchronize()
        assert e0.elapsed_time(e1) < 200.0
        assert dl.layer.last_status() == P.PRESERVE_ETIMEOUT
        assert dl.layer.last_status_code() == 6
        assert me.epoch(0) == 1 and me.epoch(1) == 1      # the rank still counts the window: it stays in step
        # the peer arrives after all
        me.debug_arrive(1, 2, FAR)
        dl.layer.clear_status()
        me.write(0, G.bits_to_cuda(t["partials_in"][rank]))
        dl.k_cache.copy_(G.bits_to_cuda(t["k_cache"]))
        dl.v_cache.copy_(G.bits_to_cuda(t["v_cache"]))
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            dl.run(stream)
        stream.synchronize()
        assert dl.layer.last_status() == P.PRESERVE_OK
        for name in ("attn_partial", "h2", "mlp_partial"):
            G.assert_close(dl.outputs()[name], ref[name], name)
    finally:
        dl.close()
        for c in comms:
            c.close()


def test_external_attention_sum_and_argument_checks(oracle):
    """The library-collective baseline's hook: window B takes a caller-reduced buffer as its partial 0.
    With the buffer holding this shard's own attention partial sums the step equals the plain one."""
    shape = I.small_shape(name="ext_sum", batch=6, ctx=80, seed=83)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t)
    dl = G.DeviceLayer(shape, t)
    try:
        dl.run()
        own = dl.attn_out.t.clone()
        dl.layer.set_external_attention_sum(own)
        dl.mlp_out.t.zero_()
        dl.run()
        assert dl.layer.last_status() == P.PRESERVE_OK
        for name in ("h2", "mlp_partial"):
            G.assert_close(dl.outputs()[name], ref[name], name)
        # a comm and an external sum exclude each other; a comm of the wrong size is refused
        c = P.Comm(0, 1, shape.batch, shape.hidden)
        try:
            with pytest.raises(P.PreserveError):
                dl.layer.set_comm(c)             # external sum still set (and n_ranks != tp_degree)
            dl.layer.set_external_attention_sum(None)
            with pytest.raises(P.PreserveError) as e:
                dl.layer.set_comm(c)
            assert e.value.code == P.PRESERVE_ESHAPE
        finally:
            c.close()
        c2 = P.Comm(1, 2, shape.batch, shape.hidden)
        try:
            with pytest.raises(P.PreserveError):
                dl.layer.set_comm(c2)            # peer 0 not connected
        finally:
            c2.close()
    finally:
        dl.close()
    import ctypes as C
    h = C.c_void_p()
    assert P.lib().preserve_comm_create(0, 9, 4, 512, C.byref(h)) == P.PRESERVE_EINVAL
    assert P.lib().preserve_comm_create(3, 2, 4, 512, C.byref(h)) == P.PRESERVE_EINVAL


def _peer_process(conn, shape_kw, a_bits, b_bits):
    """A second PROCESS on the same GPU that only owns an exchange block: it fills its two buffers,
    exports the block's handle and keeps the block alive until told to stop.  It launches no kernel
    that waits for anything."""
    import torch as _t
    from paper_2501_08192_b200 import binding as _P
    import gpu_util as _G
    _t.cuda.set_device(0)
    c = _P.Comm(1, 2, shape_kw["batch"], shape_kw["hidden"])
    c.write(0, _G.bits_to_cuda(a_bits))
    c.write(1, _G.bits_to_cuda(b_bits))
    _t.cuda.synchronize()
    conn.send(c.export_handle())
    conn.recv()                      # parent is done
    c.close()
    conn.send("closed")


def test_peer_block_of_another_process_is_read_through_its_ipc_handle(oracle):
    """The exchange block of rank 1 lives in ANOTHER PROCESS (same GPU): rank 0 maps it from the
    exported 64-byte handle, as it would map a peer GPU's block, and the fused window reads rank 1's
    partial sums through that mapping.  Rank 1's arrival is set from the host (it runs no step)."""
    import multiprocessing as mp
    import os
    import sys
    shape = I.small_shape(name="comm_ipc", batch=4, hidden=512, ffn=256, tp_degree=2, ctx=60, ctx_min=3, seed=84)
    t = I.make_layers(shape, 1)[0]
    ref = oracle.layer_step(shape, t)
    ctx = mp.get_context("spawn")
    here, there = ctx.Pipe()
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    child = ctx.Process(target=_peer_process, args=(there, dict(batch=shape.batch, hidden=shape.hidden),
                                                    t["partials_in"][1], t["attn_peer_partials"][0]))
    child.start()
    me = P.Comm(0, 2, shape.batch, shape.hidden)
    dl = G.DeviceLayer(shape, t)
    stream = torch.cuda.Stream()
    try:
        assert here.poll(120), "the peer process did not export its block"
        me.import_handle(1, here.recv())
        me.write(0, G.bits_to_cuda(t["partials_in"][0]))
        me.debug_arrive(0, 1, FAR)
        me.debug_arrive(1, 1, FAR)
        dl.layer.set_comm(me)
        with torch.cuda.stream(stream):
            dl.run(stream)
        stream.synchronize()
        assert dl.layer.last_status_code() == 0
        out = dl.outputs()
        for name in ("attn_partial", "h2", "mlp_partial"):
            G.assert_close(out[name], ref[name], name)
        # importing the same rank twice, or the own rank, is refused
        import ctypes as C
        buf = (C.c_uint8 * 64)()
        assert P.lib().preserve_comm_import(me.handle, 1, buf) == P.PRESERVE_EINVAL
        assert P.lib().preserve_comm_import(me.handle, 0, buf) == P.PRESERVE_EINVAL
    finally:
        dl.close()
        me.close()                    # unmaps the peer's block before the peer frees it
        here.send("done")
        child.join(timeout=60)
        assert child.exitcode == 0
