"""GPU operator tests through the C ABI: tensor-core GEMM and attention kernels against the CPU oracle's
definitions on sizes that span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import rel_l2, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("act", [torch.bfloat16, torch.float16])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 128, 128), (300, 512, 256), (1, 256, 64), (129, 384, 192),
                                   (1000, 4096, 4096), (2500, 1024, 512)])
def test_gemm_tcgen05(M, N, K, act):
    """A x B^T with both operands bf16 or both fp16, fp32 accumulation in tensor memory."""
    import paper_2410_03960_b200 as P
    a = S.matrix(11, 1, M, K, act, "cuda", std=1.0)
    b = S.matrix(11, 2, N, K, act, "cuda", std=1.0)
    c = P.gemm_tc(a, b)
    torch.cuda.synchronize()
    ref = to_np(a) @ to_np(b).T                      # fp64 product of the same bf16 inputs
    got = to_np(c)
    assert np.isfinite(got).all()
    # the only rounding is the final store (2^-9 relative for bf16, 2^-12 for fp16) on top of fp32 accumulation
    ulp = 2.0 ** -8 if act == torch.bfloat16 else 2.0 ** -11
    assert rel_l2(got, ref) < ulp
    assert np.max(np.abs(got - ref)) <= ulp * np.max(np.abs(ref)) + 1e-3


@pytest.mark.parametrize("M,N,K", [(200, 128, 32), (1000, 384, 4096), (77, 1024, 160), (4096, 256, 2048)])
def test_gemm_tf32_tcgen05(M, N, K):
    """fp32 operands on the tensor cores (kind::tf32): each operand enters with 10 mantissa bits, the products are summed in
    fp32.  Against the fp64 product of the fp32 inputs the error of one term is at most 2 * 2^-10 relative (two truncated or
    rounded operands); against the fp64 product of inputs whose low 13 mantissa bits are cleared it is fp32 summation noise
    if the hardware truncates -- either way bounded by the first figure, and far from a 16-bit operand's 2^-8."""
    import paper_2410_03960_b200 as P
    a = S.matrix(12, 1, M, K, torch.float32, "cuda", std=1.0)
    b = S.matrix(12, 2, N, K, torch.float32, "cuda", std=1.0)
    c = P.gemm_tf32(a, b)
    torch.cuda.synchronize()
    ref = to_np(a) @ to_np(b).T
    got = to_np(c)
    assert np.isfinite(got).all()
    assert rel_l2(got, ref) <= 1.5e-3, rel_l2(got, ref)
    # accumulate form
    c2 = P.gemm_tf32(a, b, out=c.clone())
    torch.cuda.synchronize()
    assert rel_l2(to_np(c2), 2.0 * ref) <= 1.5e-3
    # the product of the truncated inputs pins the operand handling more tightly (either rounding mode gives < 6e-4)
    def trunc(x):
        return (x.view(torch.int32) & ~0x1FFF).view(torch.float32)
    ref_t = to_np(trunc(a)) @ to_np(trunc(b)).T
    print(f"tf32 gemm {M}x{N}x{K}: rel-L2 vs exact {rel_l2(got, ref):.2e}, vs truncated operands {rel_l2(got, ref_t):.2e}")
    assert min(rel_l2(got, ref), rel_l2(got, ref_t)) <= 6e-4


@pytest.mark.parametrize("qdtype,dtype,bar", [(torch.float32, torch.float32, 1e-5), (torch.bfloat16, torch.bfloat16, 1e-2),
                                              (torch.float16, torch.bfloat16, 1e-3)])
@pytest.mark.parametrize("lens,n_q,n_kv,hd", [([5, 1, 70], 8, 2, 32), ([33, 64], 4, 4, 64), ([130], 8, 2, 128)])
def test_attention_simt(qdtype, dtype, bar, lens, n_q, n_kv, hd):
    import paper_2410_03960_b200 as P
    T = sum(lens)
    q = S.matrix(3, 1, T, n_q * hd, qdtype, "cuda", std=1.0).view(T, n_q, hd)
    k = S.matrix(3, 2, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(3, 3, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    out = P.attention_prefill(q, k, v, lens, use_tensor_cores=False)
    torch.cuda.synchronize()
    off = 0
    for n in lens:
        ref = O.causal_attention(to_np(q[off:off + n]), to_np(k[off:off + n]), to_np(v[off:off + n]))
        assert rel_l2(to_np(out[off:off + n]), ref) < bar
        off += n


@pytest.mark.parametrize("act,bar", [(torch.bfloat16, 1e-2), (torch.float16, 2.5e-3)])
@pytest.mark.parametrize("lens,n_q,n_kv", [([5, 1, 70], 8, 2), ([300, 129, 128, 1], 8, 2), ([1000], 4, 1),
                                           ([128], 2, 1), ([127, 257], 16, 2), ([2500, 700], 8, 4)])
def test_attention_tcgen05(lens, n_q, n_kv, act, bar):
    """Tensor-core flash attention (head_dim 128) against the oracle's explicit softmax(QK^T)V, prompt by prompt:
    single-tile, multi-tile, ragged and one-token prompts."""
    import paper_2410_03960_b200 as P
    hd, T = 128, sum(lens)
    q = S.matrix(5, 1, T, n_q * hd, act, "cuda", std=1.0).view(T, n_q, hd)
    k = S.matrix(5, 2, T, n_kv * hd, act, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(5, 3, T, n_kv * hd, act, "cuda", std=1.0).view(T, n_kv, hd)
    out = P.attention_prefill(q, k, v, lens, use_tensor_cores=True)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    off = 0
    for n in lens:
        ref = O.causal_attention(to_np(q[off:off + n]), to_np(k[off:off + n]), to_np(v[off:off + n]))
        got = to_np(out[off:off + n])
        # P is rounded to the activation type before the PV product and the output is stored in it
        assert rel_l2(got, ref) < bar, (n, rel_l2(got, ref))
        assert np.max(np.abs(got - ref)) < 5 * bar
        off += n


@pytest.mark.parametrize("dtype,bar", [(torch.float32, 1e-5), (torch.bfloat16, 1e-5)])
@pytest.mark.parametrize("lens,n_q,n_kv,hd", [([5, 1, 70], 8, 2, 32), ([1000, 3000, 257], 8, 2, 128), ([20000], 4, 1, 128),
                                              ([300] * 8, 32, 8, 128)])
def test_tail_attention(dtype, bar, lens, n_q, n_kv, hd):
    """One query per prompt over its cache rows, keys split across CTAs, against the oracle's definition.  The
    cache values are exactly representable (bf16 inputs are upcast), so only fp32 arithmetic separates the two."""
    import paper_2410_03960_b200 as P
    T, B = sum(lens), len(lens)
    q = S.matrix(6, 1, B, n_q * hd, torch.float32, "cuda", std=1.0).view(B, n_q, hd)
    k = S.matrix(6, 2, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(6, 3, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    out = P.tail_attention(q, k, v, lens)
    torch.cuda.synchronize()
    off = 0
    for b, n in enumerate(lens):
        ref = O.single_query_attention(to_np(q[b]), to_np(k[off:off + n]), to_np(v[off:off + n]))
        assert rel_l2(to_np(out[b]), ref) < bar
        off += n


def test_tail_attention_empty_sequence_gives_zeros_not_nan():
    """A prompt of length 0 between two ordinary ones: no key, no probability mass -- the row is zeros (not 0/0) and
    its neighbours are unaffected."""
    import paper_2410_03960_b200 as P
    lens, n_q, n_kv, hd = [40, 0, 700], 8, 2, 128
    T, B = sum(lens), len(lens)
    q = S.matrix(8, 1, B, n_q * hd, torch.float32, "cuda", std=1.0).view(B, n_q, hd)
    k = S.matrix(8, 2, T, n_kv * hd, torch.bfloat16, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(8, 3, T, n_kv * hd, torch.bfloat16, "cuda", std=1.0).view(T, n_kv, hd)
    out = P.tail_attention(q, k, v, lens)
    torch.cuda.synchronize()
    assert torch.isfinite(out).all() and (out[1] == 0).all()
    off = 0
    for b, n in enumerate(lens):
        if n:
            ref = O.single_query_attention(to_np(q[b]), to_np(k[off:off + n]), to_np(v[off:off + n]))
            assert rel_l2(to_np(out[b]), ref) < 1e-5
        off += n
