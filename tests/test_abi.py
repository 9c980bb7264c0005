"""Host-side checks of the C-ABI boundary that need no GPU: the library loads, exports every declared symbol,
and rejects bad arguments with status codes (never an exception, never an abort)."""
import ctypes as C
import os
import re

import pytest
import torch

import synthetic_inputs as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2410_03960_b200 import build, binding
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    from paper_2410_03960_b200 import binding
    header = open(os.path.join(ROOT, "include", "swiftkv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(swiftkv_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in swiftkv.h but not exported"
    assert declared == set(binding.EXPORTS)
    assert lib.swiftkv_version() >= 100


def test_workspace_bytes_validates_and_accounts_for_acrosskv(lib):
    from paper_2410_03960_b200 import SwiftKVError, workspace_bytes
    shape = S.LLAMA31_8B
    # Sec. 4: 50% SingleInputKV + g-way AcrossKV saves (L-l)/L * (1-1/g) of the cache
    _, full = workspace_bytes(shape, torch.bfloat16, 4096, 4, 32, 1)
    assert full == 32 * 2 * 4096 * 1024 * 2
    for g, saved in [(1, 0.0), (2, 0.25), (4, 0.375), (8, 0.4375), (16, 0.46875)]:
        _, kv = workspace_bytes(shape, torch.bfloat16, 4096, 4, 16, g)
        assert kv == round(full * (1 - saved))
    _, kv = workspace_bytes(shape, torch.bfloat16, 4096, 4, 29, 2)     # short last group: layers 30,31 | 32
    assert kv == (29 + 2) * 2 * 4096 * 1024 * 2
    ws1, _ = workspace_bytes(shape, torch.bfloat16, 4096, 4, 16, 1)
    ws4, _ = workspace_bytes(shape, torch.bfloat16, 4096, 4, 16, 4)
    assert ws1 - ws4 == (16 - 4) * 2 * 1024 * 4096 * 2                  # the folded weight shrinks with the groups
    for bad in [dict(max_tokens=0), dict(max_seqs=0), dict(swift_layer=0), dict(swift_layer=33), dict(acrosskv_group=0)]:
        args = dict(max_tokens=128, max_seqs=2, swift_layer=16, acrosskv_group=1)
        args.update(bad)
        with pytest.raises(SwiftKVError) as e:
            workspace_bytes(shape, torch.bfloat16, **args)
        assert e.value.code == -1
    # FP8 cache (appendix, KV quantization): one byte per element plus one fp32 scale per token row and plane; with
    # 4-way AcrossKV the paper's 68.75 % reduction against the 16-bit cache of the unmodified model (scales aside)
    from paper_2410_03960_b200 import KV_FP8
    _, kv8 = workspace_bytes(shape, torch.bfloat16, 4096, 4, 16, 4, KV_FP8)
    assert kv8 == (16 + 4) * 2 * (4096 * 1024 + 4096 * 4)
    assert abs((1 - (kv8 - (16 + 4) * 2 * 4096 * 4) / full) - 0.6875) < 1e-12
    with pytest.raises(SwiftKVError):
        workspace_bytes(shape, torch.bfloat16, 4096, 4, 16, 4, 7)       # unknown cache format
    assert lib.swiftkv_quantize_rows_fp8(None, 1, 1, None, None, None, None) == -1
    assert lib.swiftkv_tail_attention_fp8(None, None, None, None, None, None, None, 1, 1, 1, 1, 2, None, 0, None) == -1
    odd = S.ModelShape(512, 256, 4, 8, 3, 32, 688, 10000.0)
    with pytest.raises(SwiftKVError):
        workspace_bytes(odd, torch.float32, 128, 2, 2, 1)


def test_tail_attention_scratch_covers_every_shorter_maximum(lib):
    """A model's split-KV scratch is sized once from max_tokens but used with each batch's own longest sequence.  The
    split count ceil(n / chunk(n)) is not monotonic in n (chunks are whole rounds of 128 keys, at most 64 splits,
    at least 512 keys), so the size query must cover every n <= max_tokens, not just n = max_tokens."""
    def splits(n):
        c = -(-n // 64)
        c = -(-c // 128) * 128
        c = max(c, 512)
        return -(-n // c)
    assert splits(32768) == 64 and splits(33000) < 64          # the non-monotonic spot: 64 splits, then fewer
    per_split = 8 * 32 * (128 + 2) * 4
    for T in (1, 511, 512, 513, 4096, 20000, 32768, 33000, 41123, 65536, 100000, 131072):
        have = lib.swiftkv_tail_attention_scratch_bytes(8, 32, 128, T)
        assert have % per_split == 0
        worst = max(splits(n) for n in range(1, T + 1, 7)) if T > 1 else 1
        worst = max(worst, splits(T), splits(min(T, 32768)))
        assert have >= worst * per_split, (T, have // per_split, worst)
    sizes = [lib.swiftkv_tail_attention_scratch_bytes(8, 32, 128, T) for T in range(1, 70000, 97)]
    assert all(a <= b for a, b in zip(sizes, sizes[1:]))        # monotonic in the maximum length


def test_null_arguments_return_status_codes(lib):
    assert lib.swiftkv_workspace_bytes(None, 1, 1, 1, 1, None, None) == -1
    out = C.c_void_p()
    assert lib.swiftkv_model_load(None, None, None, 0, None, 0, 1, 1, C.byref(out)) == -1
    assert out.value is None
    assert lib.swiftkv_model_load(None, None, None, 0, None, 0, 1, 1, None) == -1
    assert b"null" in lib.swiftkv_last_error()
    assert lib.swiftkv_prefill(None, None, None, 1, 1, 1, None) == -1
    assert lib.swiftkv_kv_cache_view(None, 0, None) == -1
    assert lib.swiftkv_first_logits(None, None, None) == -1
    assert lib.swiftkv_status(None, None) == -1
    assert lib.swiftkv_gemm_tc(None, None, None, 1, 1, 1, 1, None) == -1
    lib.swiftkv_model_free(None)


def test_flop_model_matches_table1_linear_columns():
    """The executed-FLOP model behind the benchmark's TFLOP/s, against Table 1's per-token GEMM columns
    (K,V 2.6; Q,O 22; MLP 113 GFLOP per prefill token for Llama-3.1-70B) in the long-prompt limit."""
    from paper_2410_03960_b200 import prefill_flops
    s = S.LLAMA31_70B
    n = 1 << 20
    f = prefill_flops(s.hidden, s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.vocab, [n], s.n_layers, 1)
    assert abs(f["gemm"] / n / 1e9 - (2.68 + 21.5 + 112.7)) < 0.2
    half = prefill_flops(s.hidden, s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.ffn, s.vocab, [n], 40, 1)
    assert abs(half["gemm"] / n / 1e9 - (2.68 + 10.7 + 56.4)) < 0.2
    assert abs(half["attention"] / f["attention"] - 0.5) < 1e-9
