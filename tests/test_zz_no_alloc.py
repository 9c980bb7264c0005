"""swiftkv_tail_attention_noalloc through the C ABI: the variant of the split-KV single-query attention that keeps its
partial results in the library's built-in device array, for callers that cannot allocate device memory (a plug-in in
a process whose pool is fully committed, or code running where the allocator may not be called).

Collected last on purpose: a run that stops at the first failure has then already run every other test.
The test passes alone in a fresh process and after the other tests; it checks two calls in a row, because the
second call sees the array as the first one left it.
"""
import numpy as np
import pytest
import torch

import synthetic_inputs as S
from oracle import swiftkv_oracle as O

pytestmark = pytest.mark.gpu


def _inputs(seed, lens, n_q, n_kv, hd, dtype):
    T, B = sum(lens), len(lens)
    q = S.matrix(seed, 1, B, n_q * hd, torch.float32, "cuda", std=1.0).view(B, n_q, hd)
    k = S.matrix(seed, 2, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    v = S.matrix(seed, 3, T, n_kv * hd, dtype, "cuda", std=1.0).view(T, n_kv, hd)
    cu = torch.tensor([0] + list(torch.tensor(lens).cumsum(0)), dtype=torch.int32, device="cuda")
    return q, k, v, cu


def test_noalloc_matches_the_scratch_passing_entry_point_twice_in_a_row():
    import paper_2410_03960_b200 as P
    # first a long problem that fills many splits of the built-in array, then a shorter one with other shapes:
    # stale partials of the first call must not leak into the second
    cases = [(21, [5000, 1, 777, 12000], 32, 8, 128, torch.bfloat16), (22, [300, 45], 8, 2, 64, torch.float32)]
    for seed, lens, n_q, n_kv, hd, dtype in cases:
        q, k, v, cu = _inputs(seed, lens, n_q, n_kv, hd, dtype)
        want = P.tail_attention(q, k, v, lens)                  # existing entry point, caller-provided scratch
        out = torch.full((len(lens), n_q * hd), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        # the allocator's running count of allocations (bytes in use can also drop when the garbage collector frees
        # another test's tensors in the middle of the call)
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        P.tail_attention_noalloc(q, k, v, out, cu, max(lens))
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before   # the wrapper allocates nothing either
        torch.cuda.synchronize()
        assert torch.isfinite(out).all()
        # parity with the oracle's definition of the continuing token's attention (all keys of its prompt, softmax
        # scale 1/sqrt(hd)), prompt by prompt; the cache values are exactly representable, so only fp32 arithmetic
        # separates the two
        f64 = lambda t: t.detach().float().cpu().double().numpy()   # noqa: E731
        off = 0
        for b, n in enumerate(lens):
            ref = O.single_query_attention(f64(q[b]), f64(k[off:off + n]), f64(v[off:off + n]))
            got = f64(out[b])
            assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 1e-5, (b, n)
            off += n
        # and with the scratch-passing entry point: same kernels, same split of the keys, same arithmetic order
        assert torch.equal(out, want)


def test_noalloc_rejects_problems_beyond_the_built_in_array():
    import paper_2410_03960_b200 as P
    lib = P.load_library()
    lens = [70000] * 8                                          # 8 prompts x 64 heads x 64 splits x 130 floats > 9 MiB
    assert lib.swiftkv_tail_attention_scratch_bytes(8, 64, 128, 70000) > 9 * 1024 * 1024
    q = torch.zeros((8, 64, 128), dtype=torch.float32, device="cuda")
    kv = torch.zeros((8, 8, 128), dtype=torch.bfloat16, device="cuda")   # never read: the call is refused up front
    out = torch.zeros((8, 64 * 128), dtype=torch.float32, device="cuda")
    cu = torch.zeros(9, dtype=torch.int32, device="cuda")
    with pytest.raises(P.SwiftKVError) as e:
        P.tail_attention_noalloc(q, kv, kv, out, cu, max(lens))
    assert e.value.code == -2 and "9 MiB" in str(e.value)
    torch.cuda.synchronize()
