"""GPU operator tests through the C ABI: tensor-core GEMM and attention kernels against the CPU oracle's
definitions on sizes that span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O
from helpers import rel_l2, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 128, 128), (300, 512, 256), (1, 256, 64), (129, 384, 192),
                                   (1000, 4096, 4096), (2500, 1024, 512)])
def test_gemm_bf16_tcgen05(M, N, K):
    import paper_2410_03960_b200 as P
    a = S.matrix(11, 1, M, K, torch.bfloat16, "cuda", std=1.0)
    b = S.matrix(11, 2, N, K, torch.bfloat16, "cuda", std=1.0)
    c = P.gemm_bf16(a, b)
    torch.cuda.synchronize()
    ref = to_np(a) @ to_np(b).T                      # fp64 product of the same bf16 inputs
    got = to_np(c)
    assert np.isfinite(got).all()
    # the only rounding is the final fp32 -> bf16 store (2^-9 relative) on top of fp32 accumulation
    assert rel_l2(got, ref) < 4e-3
    assert np.max(np.abs(got - ref)) <= 2 ** -8 * np.max(np.abs(ref)) + 1e-3


@pytest.mark.parametrize("dtype,bar", [(torch.float32, 1e-5), (torch.bfloat16, 1e-2)])
@pytest.mark.parametrize("lens,n_q,n_kv,hd", [([5, 1, 70], 8, 2, 32), ([33, 64], 4, 4, 64), ([130], 8, 2, 128)])
def test_attention_simt(dtype, bar, lens, n_q, n_kv, hd):
    import paper_2410_03960_b200 as P
    T = sum(lens)
    q = S.matrix(3, 1, T, n_q * hd, dtype, "cuda", std=1.0).view(T, n_q, hd)
    k = S.matrix(3, 2, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(3, 3, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    out = P.attention_prefill(q, k, v, lens, use_tensor_cores=False)
    torch.cuda.synchronize()
    off = 0
    for n in lens:
        ref = O.causal_attention(to_np(q[off:off + n]), to_np(k[off:off + n]), to_np(v[off:off + n]))
        assert rel_l2(to_np(out[off:off + n]), ref) < bar
        off += n


@pytest.mark.parametrize("lens,n_q,n_kv", [([5, 1, 70], 8, 2), ([300, 129, 128, 1], 8, 2), ([1000], 4, 1),
                                           ([128], 2, 1), ([127, 257], 16, 2), ([2500, 700], 8, 4)])
def test_attention_tcgen05(lens, n_q, n_kv):
    """Tensor-core flash attention (head_dim 128) against the oracle's explicit softmax(QK^T)V, prompt by prompt:
    single-tile, multi-tile, ragged and one-token prompts."""
    import paper_2410_03960_b200 as P
    hd, T = 128, sum(lens)
    q = S.matrix(5, 1, T, n_q * hd, torch.bfloat16, "cuda", std=1.0).view(T, n_q, hd)
    k = S.matrix(5, 2, T, n_kv * hd, torch.bfloat16, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(5, 3, T, n_kv * hd, torch.bfloat16, "cuda", std=1.0).view(T, n_kv, hd)
    out = P.attention_prefill(q, k, v, lens, use_tensor_cores=True)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()
    off = 0
    for n in lens:
        ref = O.causal_attention(to_np(q[off:off + n]), to_np(k[off:off + n]), to_np(v[off:off + n]))
        got = to_np(out[off:off + n])
        # P is rounded to bf16 before the PV product and the output is stored in bf16
        assert rel_l2(got, ref) < 1e-2, (n, rel_l2(got, ref))
        assert np.max(np.abs(got - ref)) < 0.05
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
