"""GPU: programmatic dependent launch of the one-CTA-per-row hook kernel.  The part of the kernel that runs ahead
of its predecessor reads only library-owned tables; `hidden`, gate scores and multi-class probe weights are read
after the in-kernel wait.  These tests put the hook directly behind kernels that WRITE what it reads, inside one
captured graph, and require bit-identical results with the programmatic launch on and off."""
import numpy as np
import pytest
import torch

import workloads as W

from parity import CANARY_F32, check_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"
HOOK_BIT = 8


def _mixlib():
    import paper_2607_22595_b200 as mixlib
    return mixlib


def _canary(T, C):
    return torch.from_numpy(np.full((T, C), CANARY_F32, dtype=np.uint32).view(np.float32)).to(DEV)


def _run_chain(w, n_steps, mask, producer):
    """One graph: n_steps x ([producer kernel writing `h`] -> hook on `h` -> copy of `h` and the scores out)."""
    mixlib = _mixlib()
    old = mixlib.set_pdl_mask(-1)
    mixlib.set_pdl_mask(mask)
    try:
        m = W.make_context(mixlib.Mix, w)
        T, C = w.T_max, max(w.C_max, 1)
        g = torch.Generator(device=DEV); g.manual_seed(11)
        srcs = [(w.hidden.float() + 0.25 * i * torch.randn(w.hidden.shape, generator=g, device=DEV)).to(torch.bfloat16)
                for i in range(n_steps)]
        h = w.hidden.clone()
        scores = _canary(T, C)
        outs = [torch.empty_like(h) for _ in range(n_steps)]
        souts = [torch.empty_like(scores) for _ in range(n_steps)]
        s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            m.apply(h, scores, stream=s)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=s):
                for i in range(n_steps):
                    if producer:
                        h.copy_(srcs[i])                     # an ordinary kernel that writes what the hook reads
                    m.apply(h, scores, stream=s)
                    if producer:
                        outs[i].copy_(h)
                        souts[i].copy_(scores)
        torch.cuda.current_stream().wait_stream(s)
        h.copy_(w.hidden)
        scores.copy_(_canary(T, C))
        graph.replay()
        torch.cuda.synchronize()
        assert m.get_status() == 0
        res = dict(h=W.bits(h), scores=scores.cpu().numpy(), outs=[W.bits(o) for o in outs],
                   souts=[x.cpu().numpy() for x in souts], srcs=srcs)
        m.destroy()
        return res
    finally:
        mixlib.set_pdl_mask(old)


def test_hook_behind_a_producer_kernel_reads_fresh_rows():
    mixlib = _mixlib()
    w = W.make_decode(DEV)
    default = mixlib.set_pdl_mask(-1)
    assert default & HOOK_BIT, "the hook kernel's programmatic launch is on by default"
    a = _run_chain(w, 6, default, producer=True)
    b = _run_chain(w, 6, default & ~HOOK_BIT, producer=True)
    for i in range(6):
        assert np.array_equal(a["outs"][i], b["outs"][i]), "step %d" % i
        assert np.array_equal(a["souts"][i].view(np.uint32), b["souts"][i].view(np.uint32)), "step %d" % i
    # and both are right: step 3 against the oracle on the rows the producer wrote
    wh = W.host(w)
    wh.hidden = W.bits(a["srcs"][3])
    out = dict(hidden=a["outs"][3], scores=a["souts"][3], topk_idx=None, topk_val=None, n_active=None, status=0)
    check_parity(wh, out, check_features=False)


def test_back_to_back_hooks_accumulate_identically():
    mixlib = _mixlib()
    w = W.make_decode(DEV)
    default = mixlib.set_pdl_mask(-1)
    a = _run_chain(w, 24, default, producer=False)            # 24 hooks in a row on one buffer: steering accumulates
    b = _run_chain(w, 24, default & ~HOOK_BIT, producer=False)
    assert np.array_equal(a["h"], b["h"])
    assert np.array_equal(a["scores"].view(np.uint32), b["scores"].view(np.uint32))
    assert not np.array_equal(a["h"], W.bits(w.hidden))       # something was steered


def test_request_map_composed_by_a_kernel_is_seen_by_the_next_hook():
    """mix_set_request_map composes the slot map with a kernel; the hook enqueued right behind it must see the new
    map (the library launches that one hook the ordinary way: the map is then not a table only copies write)."""
    mixlib = _mixlib()
    w = W.make_decode(DEV)
    m = W.make_context(mixlib.Mix, w)
    T = w.T_max
    token_req = torch.arange(T, dtype=torch.int32, device=DEV)            # one request per row
    slot_a = torch.from_numpy(w.token_slot.copy()).to(DEV)
    slot_b = torch.from_numpy(np.roll(w.token_slot, 7).copy()).to(DEV)    # another assignment of apps to requests
    h = w.hidden.clone()
    scores = _canary(T, 1)
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    for slots in (slot_b, slot_a, slot_b, slot_a):
        with torch.cuda.stream(s):
            h.copy_(w.hidden)
            scores.copy_(_canary(T, 1))
            m.apply(h, scores, stream=s)                                  # a hook with the OLD map right in front
            h.copy_(w.hidden)
            scores.copy_(_canary(T, 1))
            m.set_request_map(token_req, slots, T, stream=s)
            m.apply(h, scores, stream=s)
        s.synchronize()
        wh = W.host(w)
        wh.token_slot = slots.cpu().numpy()
        out = dict(hidden=W.bits(h), scores=scores.cpu().numpy(), topk_idx=None, topk_val=None, n_active=None,
                   status=m.get_status())
        check_parity(wh, out, check_features=False)
    m.destroy()


def _run_sae_calls(w, n_calls, mask, flags=0):
    """One graph: n_calls x (copy a fresh batch into `h` -> mix_apply -> copy `h` out); returns the bits of every result."""
    mixlib = _mixlib()
    old = mixlib.set_pdl_mask(-1)
    mixlib.set_pdl_mask(mask)
    try:
        m = W.make_context(mixlib.Mix, w, flags=flags)
        T, C = w.T_max, max(w.C_max, 1)
        g = torch.Generator(device=DEV); g.manual_seed(5)
        srcs = [(w.hidden.float() * (1.0 + 0.125 * i) + 0.125 * i * torch.randn(w.hidden.shape, generator=g, device=DEV)).to(torch.bfloat16)
                for i in range(n_calls)]
        h = w.hidden.clone()
        scores = _canary(T, C)
        outs = [torch.empty_like(h) for _ in range(n_calls)]
        souts = [torch.empty_like(scores) for _ in range(n_calls)]
        s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            m.apply(h, scores, stream=s)
            scores.copy_(_canary(T, C))
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=s):
                for i in range(n_calls):
                    h.copy_(srcs[i])
                    m.apply(h, scores, stream=s)
                    outs[i].copy_(h)
                    souts[i].copy_(scores)
        torch.cuda.current_stream().wait_stream(s)
        for _ in range(2):                                   # the second replay starts from the first one's device state
            graph.replay()
        torch.cuda.synchronize()
        assert m.get_status() == 0
        res = [(W.bits(o), x.cpu().numpy()) for o, x in zip(outs, souts)]
        m.destroy()
        return res, srcs
    finally:
        mixlib.set_pdl_mask(old)


@pytest.mark.parametrize("make", ["tiny", "small_mixed"])
def test_sae_chain_is_bit_identical_with_programmatic_launches_on_and_off(make):
    """The SAE chain's kernels (front -> encode -> tail -> fallback pair) start early under programmatic launch and
    wait inside; back-to-back calls in one graph reuse every workspace of the context.  Same bits either way, and
    right against the oracle."""
    mixlib = _mixlib()
    w = W.make_tiny(DEV) if make == "tiny" else W.make_mixed(DEV, T=1024, d=512, d_sae=2048, R=16)
    default = mixlib.set_pdl_mask(-1)
    assert default & 2 and default & 4, "encode and tail are launched programmatically by default"
    a, srcs = _run_sae_calls(w, 3, default)
    b, _ = _run_sae_calls(w, 3, 0)
    for i in range(3):
        assert np.array_equal(a[i][0], b[i][0]), "call %d" % i
        assert np.array_equal(a[i][1].view(np.uint32), b[i][1].view(np.uint32)), "call %d" % i
    wh = W.host(w)
    wh.hidden = W.bits(srcs[2])
    out = dict(hidden=a[2][0], scores=a[2][1], topk_idx=None, topk_val=None, n_active=None, status=0)
    check_parity(wh, out, check_features=False)
