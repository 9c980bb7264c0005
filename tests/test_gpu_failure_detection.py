"""What the library reports when something goes wrong on the device -- without ever faulting, trapping or hanging a GPU:
a bounded in-kernel wait that runs out (short limit, a barrier nobody completes), and a value that does not fit the
IEEE-half activation format."""
import pytest
import torch

import synthetic_inputs as S

pytestmark = pytest.mark.gpu

MID = S.ModelShape(1024, 512, 4, 8, 2, 128, 1024, 500000.0, 1e-5, "mid")


def _model(shape, w, lens, l=2, g=1):
    import paper_2410_03960_b200 as P
    return P.SwiftKVModel(shape, w, torch.bfloat16, sum(lens), len(lens), l, g)


def test_bounded_wait_runs_out_and_is_reported_once():
    """A CTA role waits, with the kernels' own bounded wait and a limit of one million clocks (well under a millisecond),
    on a barrier that is never completed.  It must give up at its limit, the CTA's other role must leave through the
    abort flag (not by its own multi-second limit), the kernel must return, swiftkv_status must say DEVICE_TIMEOUT
    exactly once, and the model must keep working afterwards."""
    import paper_2410_03960_b200 as P
    lens = [70, 9]
    w = S.make_weights(MID, 3, torch.bfloat16, "cuda")
    tok = S.make_prompts(3, lens, MID.vocab)
    model = _model(MID, w, lens)
    model.prefill(tok, lens, 2, 1)
    model.status()
    want = model.first_logits().clone()
    gave_up, aborted = model.debug_bounded_wait(1_000_000)
    assert gave_up and aborted
    with pytest.raises(P.SwiftKVError) as e:
        model.status()
    assert e.value.code == -5
    model.status()                                   # the word was cleared by the read
    model.prefill(tok, lens, 2, 1)                   # the context and the model are still usable
    model.status()
    assert torch.equal(model.first_logits(), want)
    with pytest.raises(P.SwiftKVError) as e:
        model.debug_bounded_wait(10 ** 12)           # limits beyond ~50 ms are refused on the host
    assert e.value.code == -1
    model.close()


def test_fused_launch_grid_barrier_runs_out_and_is_reported():
    """The persistent cooperative launch of the last-token path waits at its own grid barrier and ring barriers; all are
    bounded.  A launch whose barrier cannot complete (the host claims an arrival that never happened), with a limit of one
    million clocks: every CTA gives up, the kernel returns, DEVICE_TIMEOUT is reported once, and the next prefill -- which
    uses the same kernel with the default limit -- gives the same bits as before."""
    import paper_2410_03960_b200 as P
    lens = [70, 9, 300]
    w = S.make_weights(MID, 6, torch.bfloat16, "cuda")
    tok = S.make_prompts(6, lens, MID.vocab)
    model = _model(MID, w, lens)
    assert model.set_kernel_mask(119) == 119
    model.prefill(tok, lens, 2, 1)
    model.status()
    want = model.first_logits().clone()
    model.debug_fused_barrier_wait(1_000_000)
    with pytest.raises(P.SwiftKVError) as e:
        model.status()
    assert e.value.code == -5
    model.status()
    for _ in range(2):
        model.prefill(tok, lens, 2, 1)
        model.status()
        assert torch.equal(model.first_logits(), want)
    with pytest.raises(P.SwiftKVError) as e:
        model.debug_fused_barrier_wait(10 ** 12)
    assert e.value.code == -1
    model.close()


@pytest.mark.parametrize("mask", [55, 0])
def test_half_activation_overflow_is_reported_not_silent(mask):
    """With IEEE-half activations a value beyond +-65504 is clamped -- and reported: one layer's up-projection is scaled
    so that the SwiGLU output exceeds the half range (tensor-core and SIMT kernels alike).  The same weights with
    bfloat16 activations run clean."""
    import paper_2410_03960_b200 as P
    lens = [200, 31]
    w = S.make_weights(MID, 4, torch.bfloat16, "cuda")
    w.layers[1]["w_up"] = (w.layers[1]["w_up"].float() * 3.0e5).to(torch.bfloat16)
    tok = S.make_prompts(4, lens, MID.vocab)
    model = _model(MID, w, lens)
    model.set_kernel_mask(mask)
    model.set_activation_format(P.ACT_F16)
    model.prefill(tok, lens, 2, 1)
    with pytest.raises(P.SwiftKVError) as e:
        model.status()
    assert e.value.code == -8 and "SWIFTKV_ACT_BF16" in str(e.value)
    model.set_activation_format(P.ACT_BF16)
    model.prefill(tok, lens, 2, 1)
    model.status()                                   # no clamping in bfloat16: status OK
    assert torch.isfinite(model.first_logits()).all()
    model.close()
    # and an ordinary model never raises the flag
    w2 = S.make_weights(MID, 4, torch.bfloat16, "cuda")
    m2 = _model(MID, w2, lens)
    m2.set_kernel_mask(mask)
    m2.prefill(tok, lens, 2, 1)
    m2.status()
    m2.close()
