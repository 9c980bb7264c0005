"""ctypes binding of libswiftkv.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB: Optional[C.CDLL] = None

DTYPE_F32, DTYPE_BF16, DTYPE_F16, DTYPE_FP8_E4M3 = 0, 1, 2, 3
ACT_BF16, ACT_F16, ACT_F16_SPLIT = 0, 1, 2
SPLIT_QKV_INPUT, SPLIT_SCORES, SPLIT_ATTN_OUT, SPLIT_MLP_INPUT, SPLIT_MLP_ACT = 1, 2, 4, 8, 16
KV_MODEL_DTYPE, KV_FP8 = 0, 1
_DTYPE_CODE = {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}
KC_NAMES = ("gemm", "attention", "elementwise", "tail", "gemm_swiglu")

# every symbol include/swiftkv.h declares
EXPORTS = (
    "swiftkv_version", "swiftkv_last_error", "swiftkv_workspace_bytes", "swiftkv_model_load", "swiftkv_prefill",
    "swiftkv_prefill_device_tokens", "swiftkv_step", "swiftkv_kv_cache_view", "swiftkv_first_logits", "swiftkv_status",
    "swiftkv_profile_enable", "swiftkv_profile_read", "swiftkv_last_launch_count", "swiftkv_set_kernel_mask",
    "swiftkv_set_activation_format", "swiftkv_model_free", "swiftkv_gemm_tc", "swiftkv_attention_prefill", "swiftkv_tail_attention_scratch_bytes",
    "swiftkv_tail_attention", "swiftkv_tail_attention_noalloc", "swiftkv_quantize_rows_fp8", "swiftkv_tail_attention_fp8",
    "swiftkv_debug_bounded_wait", "swiftkv_op_status", "swiftkv_set_split_mask",
    "swiftkv_gemm_tc_split", "swiftkv_attention_prefill_split", "swiftkv_simscore_scratch_bytes", "swiftkv_simscore",
    "swiftkv_distill_workspace_bytes", "swiftkv_distill_grads", "swiftkv_debug_fused_barrier_wait", "swiftkv_adamw_update", "swiftkv_gemm_tf32",
    "swiftkv_half_weight_cache_bytes", "swiftkv_set_half_weight_cache",
)


DISTILL_FP32, DISTILL_TF32X3, DISTILL_TF32 = 0, 1, 2


class SwiftKVError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"swiftkv error {code}: {msg}")
        self.code = code


class _Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("vocab", "hidden", "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "ffn")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32), ("kv_format", C.c_int32)]


class _LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("in_norm", "wq", "wk", "wv", "wo", "post_norm", "w_gate", "w_up", "w_down")]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("layers", C.POINTER(_LayerWeights))]


class _SeqStep(C.Structure):
    _fields_ = [("n_new", C.c_int32), ("n_past", C.c_int32), ("cache_row", C.c_int32), ("emit", C.c_int32),
                ("block_table", C.POINTER(C.c_int32)), ("n_blocks", C.c_int32)]


class _KVView(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
                ("token_stride", C.c_int64), ("head_stride", C.c_int64),
                ("n_tokens", C.c_int32), ("dtype", C.c_int32), ("owner_layer", C.c_int32)]


def library_path() -> str:
    return os.path.join(_HERE, "libswiftkv.so")


def load_library() -> C.CDLL:
    """Loads libswiftkv.so.  There is no fallback: without the built CUDA library nothing in this package runs."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2410_03960_b200.build` "
                           "(the SwiftKV prefill path has no CPU or PyTorch fallback)")
    lib = C.CDLL(path)
    lib.swiftkv_last_error.restype = C.c_char_p
    lib.swiftkv_workspace_bytes.argtypes = [C.POINTER(_Config), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                            C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.swiftkv_model_load.argtypes = [C.POINTER(_Config), C.POINTER(_Weights), C.c_void_p, C.c_size_t, C.c_void_p,
                                       C.c_size_t, C.c_int32, C.c_int32, C.POINTER(C.c_void_p)]
    lib.swiftkv_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.swiftkv_prefill_device_tokens.argtypes = lib.swiftkv_prefill.argtypes
    lib.swiftkv_step.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(_SeqStep), C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.swiftkv_kv_cache_view.argtypes = [C.c_void_p, C.c_int32, C.POINTER(_KVView)]
    lib.swiftkv_first_logits.argtypes = [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int32)]
    lib.swiftkv_status.argtypes = [C.c_void_p, C.c_void_p]
    lib.swiftkv_profile_enable.argtypes = [C.c_void_p, C.c_int32]
    lib.swiftkv_profile_read.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.swiftkv_last_launch_count.argtypes = [C.c_void_p]
    lib.swiftkv_set_kernel_mask.argtypes = [C.c_void_p, C.c_int32]
    lib.swiftkv_model_free.argtypes = [C.c_void_p]
    lib.swiftkv_model_free.restype = None
    lib.swiftkv_set_activation_format.argtypes = [C.c_void_p, C.c_int32]
    lib.swiftkv_set_split_mask.argtypes = [C.c_void_p, C.c_int32]
    lib.swiftkv_half_weight_cache_bytes.argtypes = [C.c_void_p, C.c_int32]
    lib.swiftkv_half_weight_cache_bytes.restype = C.c_int64
    lib.swiftkv_set_half_weight_cache.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
    lib.swiftkv_simscore_scratch_bytes.argtypes = [C.c_void_p, C.c_int32]
    lib.swiftkv_simscore_scratch_bytes.restype = C.c_size_t
    lib.swiftkv_simscore.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p,
                                     C.c_void_p]
    lib.swiftkv_distill_workspace_bytes.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
    lib.swiftkv_distill_workspace_bytes.restype = C.c_size_t
    lib.swiftkv_distill_grads.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_int32] + [C.c_void_p] * 8 + \
        [C.c_size_t, C.c_void_p]
    lib.swiftkv_gemm_tc_split.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.swiftkv_attention_prefill_split.argtypes = [C.c_void_p] * 6 + [C.c_int32, C.c_void_p] + [C.c_int32] * 6 + [C.c_void_p]
    lib.swiftkv_gemm_tc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.swiftkv_attention_prefill.argtypes = [C.c_void_p] * 5 + [C.c_int32] * 9 + [C.c_void_p]
    lib.swiftkv_gemm_tf32.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.swiftkv_adamw_update.argtypes = [C.c_void_p] * 4 + [C.c_int64, C.c_int32] + [C.c_float] * 5 + [C.c_void_p]
    lib.swiftkv_debug_fused_barrier_wait.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
    lib.swiftkv_debug_bounded_wait.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int32), C.c_void_p]
    lib.swiftkv_op_status.argtypes = [C.c_void_p]
    lib.swiftkv_tail_attention_scratch_bytes.argtypes = [C.c_int32] * 4
    lib.swiftkv_tail_attention_scratch_bytes.restype = C.c_size_t
    lib.swiftkv_tail_attention.argtypes = [C.c_void_p] * 5 + [C.c_int32] * 6 + [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.swiftkv_tail_attention_noalloc.argtypes = [C.c_void_p] * 5 + [C.c_int32] * 6 + [C.c_void_p]
    lib.swiftkv_quantize_rows_fp8.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.swiftkv_tail_attention_fp8.argtypes = [C.c_void_p] * 7 + [C.c_int32] * 5 + [C.c_void_p, C.c_size_t, C.c_void_p]
    _LIB = lib
    return lib


def _check(rc: int) -> None:
    if rc != 0:
        raise SwiftKVError(rc, load_library().swiftkv_last_error().decode())


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _make_config(shape, dtype: torch.dtype, kv_format: int = KV_MODEL_DTYPE) -> _Config:
    code = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[dtype]
    return _Config(shape.vocab, shape.hidden, shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                   shape.ffn, float(shape.rope_theta), float(shape.rms_eps), code, kv_format)


def workspace_bytes(shape, dtype: torch.dtype, max_tokens: int, max_seqs: int, swift_layer: int,
                    acrosskv_group: int, kv_format: int = KV_MODEL_DTYPE) -> Tuple[int, int]:
    """swiftkv_workspace_bytes -> (workspace_bytes, kv_cache_bytes)."""
    cfg = _make_config(shape, dtype, kv_format)
    ws, kv = C.c_size_t(0), C.c_size_t(0)
    _check(load_library().swiftkv_workspace_bytes(C.byref(cfg), max_tokens, max_seqs, swift_layer, acrosskv_group,
                                                  C.byref(ws), C.byref(kv)))
    return ws.value, kv.value


class SwiftKVModel:
    """swiftkv_model_load / swiftkv_prefill / swiftkv_kv_cache_view / swiftkv_first_logits over torch CUDA tensors.

    `weights` needs .embed, .final_norm, .lm_head and .layers (a list of dicts with in_norm, wq, wk, wv, wo,
    post_norm, w_gate, w_up, w_down) as contiguous CUDA tensors of `dtype`, [out_features, in_features].
    The workspace and the KV cache are torch tensors owned by this object.
    """

    def __init__(self, shape, weights, dtype: torch.dtype, max_tokens: int, max_seqs: int, swift_layer: int,
                 acrosskv_group: int = 1, device: str = "cuda:0", kv_format: int = KV_MODEL_DTYPE):
        self.lib = load_library()
        self.shape, self.dtype, self.device = shape, dtype, torch.device(device)
        self.kv_format = kv_format
        self.max_tokens, self.max_seqs = max_tokens, max_seqs
        self._weights = weights           # keep the tensors alive: the library borrows their memory
        ws_b, kv_b = workspace_bytes(shape, dtype, max_tokens, max_seqs, swift_layer, acrosskv_group, kv_format)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(ws_b, dtype=torch.uint8, device=self.device)
            self.kv_cache = torch.empty(kv_b, dtype=torch.uint8, device=self.device)
            cfg = _make_config(shape, dtype, kv_format)
            arr = (_LayerWeights * shape.n_layers)()
            for j, lw in enumerate(weights.layers):
                for name, _ in _LayerWeights._fields_:
                    t = lw[name]
                    assert t.is_cuda and t.is_contiguous() and t.dtype == dtype, name
                    setattr(arr[j], name, t.data_ptr())
            for t in (weights.embed, weights.final_norm, weights.lm_head):
                assert t.is_cuda and t.is_contiguous() and t.dtype == dtype
            w = _Weights(weights.embed.data_ptr(), weights.final_norm.data_ptr(), weights.lm_head.data_ptr(), arr)
            handle = C.c_void_p()
            _check(self.lib.swiftkv_model_load(C.byref(cfg), C.byref(w), self.workspace.data_ptr(), ws_b,
                                               self.kv_cache.data_ptr(), kv_b, max_tokens, max_seqs, C.byref(handle)))
        self._h = handle

    def close(self) -> None:
        if getattr(self, "_h", None):
            self.lib.swiftkv_model_free(self._h)
            self._h = None

    __del__ = close

    def prefill(self, tokens, seq_lens: Sequence[int], swift_layer: int, acrosskv_group: int = 1,
                stream: Optional[torch.cuda.Stream] = None) -> None:
        """swiftkv_prefill: `tokens` is a HOST int32 tensor (packed, prompt-major)."""
        tokens = torch.as_tensor(tokens, dtype=torch.int32).contiguous()
        assert not tokens.is_cuda
        lens = (C.c_int32 * len(seq_lens))(*[int(n) for n in seq_lens])
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_prefill(self._h, tokens.data_ptr(), lens, len(seq_lens), swift_layer, acrosskv_group,
                                            _stream_ptr(stream)))

    def prefill_device_tokens(self, tokens_dev: torch.Tensor, seq_lens: Sequence[int], swift_layer: int,
                              acrosskv_group: int = 1, stream: Optional[torch.cuda.Stream] = None) -> None:
        assert tokens_dev.is_cuda and tokens_dev.dtype == torch.int32 and tokens_dev.is_contiguous()
        lens = (C.c_int32 * len(seq_lens))(*[int(n) for n in seq_lens])
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_prefill_device_tokens(self._h, tokens_dev.data_ptr(), lens, len(seq_lens), swift_layer,
                                                          acrosskv_group, _stream_ptr(stream)))

    def step(self, tokens, seqs: Sequence[Tuple[int, int, int, int]], swift_layer: int, acrosskv_group: int = 1,
             stream: Optional[torch.cuda.Stream] = None) -> None:
        """swiftkv_step: one forward pass over a mixed minibatch.  `tokens`: HOST int32, the new tokens of all sequences
        packed in order; `seqs`: one (n_new, n_past, cache_row, emit) tuple per sequence, or -- paged cache --
        (n_new, n_past, block_table, emit) with block_table a list of 128-row page numbers."""
        tokens = torch.as_tensor(tokens, dtype=torch.int32).contiguous()
        assert not tokens.is_cuda and tokens.numel() == sum(s[0] for s in seqs)
        keep = []                      # ctypes arrays of the block tables must outlive the call
        items = []
        for a, p, r, e in seqs:
            if isinstance(r, (list, tuple)):
                tab = (C.c_int32 * len(r))(*[int(x) for x in r])
                keep.append(tab)
                items.append(_SeqStep(int(a), int(p), 0, int(e), tab, len(r)))
            else:
                items.append(_SeqStep(int(a), int(p), int(r), int(e), None, 0))
        arr = (_SeqStep * len(seqs))(*items)
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_step(self._h, tokens.data_ptr(), arr, len(seqs), swift_layer, acrosskv_group,
                                         _stream_ptr(stream)))

    def kv_cache_view(self, layer: int) -> Tuple[torch.Tensor, torch.Tensor, int]:
        """swiftkv_kv_cache_view -> (K [n_tokens, n_kv, hd], V, owner_layer) as views into the cache tensor."""
        v = _KVView()
        _check(self.lib.swiftkv_kv_cache_view(self._h, layer, C.byref(v)))
        assert v.dtype != DTYPE_FP8_E4M3, "FP8 cache: use kv_cache_view_fp8"
        flat = self.kv_cache.view(self.dtype)
        es = flat.element_size()
        n = v.n_tokens * v.token_stride
        shape = (v.n_tokens, self.shape.n_kv_heads, self.shape.head_dim)
        ko = (v.k - self.kv_cache.data_ptr()) // es
        vo = (v.v - self.kv_cache.data_ptr()) // es
        return flat[ko:ko + n].view(shape), flat[vo:vo + n].view(shape), v.owner_layer

    def kv_cache_view_fp8(self, layer: int):
        """swiftkv_kv_cache_view of an FP8 cache -> (K codes uint8 [n_tokens, n_kv, hd], V codes, K scales fp32
        [n_tokens], V scales, owner_layer) as views into the cache tensor."""
        v = _KVView()
        _check(self.lib.swiftkv_kv_cache_view(self._h, layer, C.byref(v)))
        assert v.dtype == DTYPE_FP8_E4M3
        base = self.kv_cache.data_ptr()
        n = v.n_tokens * v.token_stride
        shape = (v.n_tokens, self.shape.n_kv_heads, self.shape.head_dim)

        def codes(ptr):
            return self.kv_cache[ptr - base: ptr - base + n].view(shape)

        def scales(ptr):
            return self.kv_cache[ptr - base: ptr - base + 4 * v.n_tokens].view(torch.float32)

        return codes(v.k), codes(v.v), scales(v.k_scale), scales(v.v_scale), v.owner_layer

    def first_logits(self) -> torch.Tensor:
        """swiftkv_first_logits -> fp32 [n_seqs, vocab] view into the workspace."""
        p, n = C.c_void_p(), C.c_int32()
        _check(self.lib.swiftkv_first_logits(self._h, C.byref(p), C.byref(n)))
        off = (p.value - self.workspace.data_ptr()) // 4
        flat = self.workspace[: (self.workspace.numel() // 4) * 4].view(torch.float32)
        return flat[off: off + n.value * self.shape.vocab].view(n.value, self.shape.vocab)

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_status(self._h, _stream_ptr(stream)))

    def simscore(self, tokens, seq_lens: Sequence[int], stream: Optional[torch.cuda.Stream] = None):
        """swiftkv_simscore (Eq. 1): returns (SimScore fp32 [n_layers - 1], Similarity matrix fp32 [n_layers, n_layers])."""
        tokens = torch.as_tensor(tokens, dtype=torch.int32).contiguous()
        assert not tokens.is_cuda
        L = self.shape.n_layers
        lens = (C.c_int32 * len(seq_lens))(*[int(n) for n in seq_lens])
        nbytes = self.lib.swiftkv_simscore_scratch_bytes(self._h, int(sum(seq_lens)))
        scratch = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        sim = torch.empty((L, L), dtype=torch.float32, device=self.device)
        score = torch.empty(L - 1, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_simscore(self._h, tokens.data_ptr(), lens, len(seq_lens), scratch.data_ptr(), nbytes,
                                             sim.data_ptr(), score.data_ptr(), _stream_ptr(stream)))
            torch.cuda.current_stream().synchronize() if stream is None else stream.synchronize()
        return score, sim

    def debug_fused_barrier_wait(self, limit_clocks: int, stream: Optional[torch.cuda.Stream] = None) -> None:
        """swiftkv_debug_fused_barrier_wait: makes the fused last-token launch's grid barrier run out; status() raises afterwards."""
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_debug_fused_barrier_wait(self._h, int(limit_clocks), _stream_ptr(stream)))

    def distill_grads(self, tokens, seq_lens: Sequence[int], swift_layer: int, acrosskv_group: int, temperature: float,
                      student: dict, stream: Optional[torch.cuda.Stream] = None, precision: int = 0):
        """swiftkv_distill_grads (Sec. 3.4, Eq. 3).  student: {"wq" | "wk" | "wv": list over layers of fp32 CUDA tensors (None for
        layers <= swift_layer)}; precision: DISTILL_FP32 / DISTILL_TF32X3 / DISTILL_TF32.  Returns (loss tensor [1], {"wq" | "wk" | "wv": list of gradient tensors, None likewise})."""
        L = self.shape.n_layers
        tokens = torch.as_tensor(tokens, dtype=torch.int32).contiguous().to(self.device)
        lens = (C.c_int32 * len(seq_lens))(*[int(n) for n in seq_lens])
        nbytes = self.lib.swiftkv_distill_workspace_bytes(self._h, int(sum(seq_lens)), int(swift_layer))
        ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        loss = torch.zeros(1, dtype=torch.float32, device=self.device)
        grads = {k: [None if student[k][j] is None else torch.empty_like(student[k][j]) for j in range(L)] for k in ("wq", "wk", "wv")}

        def ptrs(lst):
            return (C.c_void_p * L)(*[None if t is None else t.data_ptr() for t in lst])
        for k in ("wq", "wk", "wv"):
            for t in student[k]:
                assert t is None or (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous())
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_distill_grads(self._h, tokens.data_ptr(), lens, len(seq_lens), int(swift_layer), int(acrosskv_group),
                                                  float(temperature), int(precision), ptrs(student["wq"]), ptrs(student["wk"]), ptrs(student["wv"]),
                                                  ptrs(grads["wq"]), ptrs(grads["wk"]), ptrs(grads["wv"]), loss.data_ptr(),
                                                  ws.data_ptr(), nbytes, _stream_ptr(stream)))
            torch.cuda.current_stream().synchronize() if stream is None else stream.synchronize()
        return loss, grads

    def debug_bounded_wait(self, limit_clocks: int, stream: Optional[torch.cuda.Stream] = None) -> Tuple[bool, bool]:
        """swiftkv_debug_bounded_wait: (the waiting role gave up at its limit, the second role left through the abort flag)."""
        out = (C.c_int32 * 2)()
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_debug_bounded_wait(self._h, int(limit_clocks), out, _stream_ptr(stream)))
        return bool(out[0]), bool(out[1])

    def profile_enable(self, on: bool) -> None:
        _check(self.lib.swiftkv_profile_enable(self._h, int(on)))

    def profile_read(self, stream: Optional[torch.cuda.Stream] = None) -> Dict[str, Tuple[float, int]]:
        ms = (C.c_float * len(KC_NAMES))()
        cnt = (C.c_int32 * len(KC_NAMES))()
        with torch.cuda.device(self.device):
            _check(self.lib.swiftkv_profile_read(self._h, _stream_ptr(stream), ms, cnt))
        return {k: (float(ms[i]), int(cnt[i])) for i, k in enumerate(KC_NAMES)}

    def last_launch_count(self) -> int:
        return int(self.lib.swiftkv_last_launch_count(self._h))

    def set_kernel_mask(self, mask: int) -> int:
        return int(self.lib.swiftkv_set_kernel_mask(self._h, mask))

    def set_activation_format(self, fmt: int) -> None:
        """swiftkv_set_activation_format: ACT_F16 (default), ACT_BF16 or ACT_F16_SPLIT (half pairs)."""
        _check(self.lib.swiftkv_set_activation_format(self._h, fmt))

    def set_split_mask(self, mask: int) -> None:
        """swiftkv_set_split_mask: which operands travel as half pairs (SPLIT_* bits)."""
        _check(self.lib.swiftkv_set_split_mask(self._h, mask))

    def set_half_weight_cache(self, n_layers: int) -> int:
        """swiftkv_set_half_weight_cache: room (a torch tensor owned by this object) for the half copies of the first
        `n_layers` layers' matrices, made once and kept from step to step; 0 removes it.  Call again after changing the
        model's weights.  Returns the bytes held."""
        cfg = _make_config(self.shape, self.dtype, self.kv_format)
        need = int(self.lib.swiftkv_half_weight_cache_bytes(C.byref(cfg), n_layers))
        if need < 0:
            raise SwiftKVError(-1, "swiftkv_half_weight_cache_bytes rejected the config")
        with torch.cuda.device(self.device):
            self._w16_cache = torch.empty(need, dtype=torch.uint8, device=self.device) if need else None
            _check(self.lib.swiftkv_set_half_weight_cache(self._h, self._w16_cache.data_ptr() if need else None, need))
        return need


def adamw_update(param: torch.Tensor, grad: torch.Tensor, exp_avg: torch.Tensor, exp_avg_sq: torch.Tensor, step: int,
                 lr: float = 3e-4, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.05,
                 stream: Optional[torch.cuda.Stream] = None) -> None:
    """swiftkv_adamw_update: one in-place AdamW step on an fp32 CUDA tensor (defaults: the paper's lr and weight decay)."""
    for t in (param, grad, exp_avg, exp_avg_sq):
        assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() == param.numel()
    with torch.cuda.device(param.device):
        _check(load_library().swiftkv_adamw_update(param.data_ptr(), grad.data_ptr(), exp_avg.data_ptr(), exp_avg_sq.data_ptr(),
                                                  param.numel(), int(step), lr, beta1, beta2, eps, weight_decay, _stream_ptr(stream)))


def split_halves(x: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """fp32 tensor -> (hi, lo) IEEE halves with hi + lo ~ x (marshalling of the half-pair operand format)."""
    hi = x.to(torch.float16)
    return hi, (x - hi.float()).to(torch.float16)


def gemm_tc_split(a: torch.Tensor, b: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_gemm_tc_split: a fp32 [M, K] (sent as half pairs), b IEEE half [N, K] -> fp32 [M, N]."""
    assert a.is_cuda and a.dtype == torch.float32 and b.dtype == torch.float16
    hi, lo = split_halves(a)
    a2 = torch.cat([hi, lo], dim=1).contiguous()
    c = torch.zeros((a.shape[0], b.shape[0]), dtype=torch.float32, device=a.device)
    with torch.cuda.device(a.device):
        _check(load_library().swiftkv_gemm_tc_split(a2.data_ptr(), b.contiguous().data_ptr(), c.data_ptr(), a.shape[0],
                                                    b.shape[0], a.shape[1], _stream_ptr(stream)))
    return c


def attention_prefill_split(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_lens: Sequence[int], out_split: bool = False,
                            stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_attention_prefill_split: q fp32 [T, n_q, hd], k fp32 [T, n_kv, hd] (sent as half pairs), v IEEE half.
    Returns fp32 [T, n_q*hd]: the half output, or hi + lo of the pair output when out_split."""
    T, n_q, hd = q.shape
    n_kv = k.shape[1]
    qh, ql = split_halves(q.contiguous())
    kh, kl = split_halves(k.contiguous())
    cu = _cu_seqlens(seq_lens, q.device)
    out = torch.zeros((T, (2 if out_split else 1) * n_q * hd), dtype=torch.float16, device=q.device)
    with torch.cuda.device(q.device):
        _check(load_library().swiftkv_attention_prefill_split(qh.data_ptr(), ql.data_ptr(), kh.data_ptr(), kl.data_ptr(),
                                                              v.contiguous().data_ptr(), out.data_ptr(), int(out_split),
                                                              cu.data_ptr(), len(seq_lens), T, max(seq_lens), n_q, n_kv, hd,
                                                              _stream_ptr(stream)))
    if out_split:
        return out[:, :n_q * hd].float() + out[:, n_q * hd:].float()
    return out.float()


def gemm_tf32(a: torch.Tensor, b: torch.Tensor, out: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_gemm_tf32: a [M, K] x b [N, K]^T with fp32 operands on the tensor cores; `out` given: accumulated into."""
    assert a.is_cuda and b.is_cuda and a.dtype == b.dtype == torch.float32 and a.is_contiguous() and b.is_contiguous()
    M, K = a.shape
    N = b.shape[0]
    acc = out is not None
    c = out if acc else torch.empty((M, N), dtype=torch.float32, device=a.device)
    with torch.cuda.device(a.device):
        _check(load_library().swiftkv_gemm_tf32(a.data_ptr(), b.data_ptr(), c.data_ptr(), M, N, K, int(acc), _stream_ptr(stream)))
    return c


def gemm_tc(a: torch.Tensor, b: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_gemm_tc: C = A @ B.T with A [M, K], B [N, K] CUDA tensors, both bf16 or both fp16; C has their dtype."""
    assert a.is_cuda and b.is_cuda and b.dtype == a.dtype and a.dtype in (torch.bfloat16, torch.float16)
    assert a.is_contiguous() and b.is_contiguous()
    m, k = a.shape
    n = b.shape[0]
    c = torch.empty((m, n), dtype=a.dtype, device=a.device)
    with torch.cuda.device(a.device):
        _check(load_library().swiftkv_gemm_tc(a.data_ptr(), b.data_ptr(), c.data_ptr(), m, n, k, _DTYPE_CODE[a.dtype],
                                              _stream_ptr(stream)))
    return c


def attention_prefill(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, seq_lens: Sequence[int],
                      use_tensor_cores: bool, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_attention_prefill on packed prompts: q [T, n_q, hd], k/v [T, n_kv, hd] -> [T, n_q*hd]."""
    assert q.is_cuda and q.is_contiguous() and k.is_contiguous() and v.is_contiguous()
    t, n_q, hd = q.shape
    n_kv = k.shape[1]
    cu = [0]
    for n in seq_lens:
        cu.append(cu[-1] + int(n))
    assert cu[-1] == t
    cu_dev = torch.tensor(cu, dtype=torch.int32, device=q.device)
    out = torch.empty((t, n_q * hd), dtype=q.dtype, device=q.device)
    with torch.cuda.device(q.device):
        _check(load_library().swiftkv_attention_prefill(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                                        cu_dev.data_ptr(), len(seq_lens), t, max(seq_lens), n_q, n_kv, hd,
                                                        _DTYPE_CODE[q.dtype], _DTYPE_CODE[k.dtype], int(use_tensor_cores),
                                                        _stream_ptr(stream)))
    return out


def _cu_seqlens(seq_lens: Sequence[int], device) -> torch.Tensor:
    cu = [0]
    for n in seq_lens:
        cu.append(cu[-1] + int(n))
    return torch.tensor(cu, dtype=torch.int32, device=device)


def tail_attention(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, seq_lens: Sequence[int],
                   stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_tail_attention: q fp32 [n_seqs, n_q, hd]; caches [T, n_kv, hd] (bf16 or fp32) -> fp32 [n_seqs, n_q*hd]."""
    assert q.is_cuda and q.dtype == torch.float32 and q.is_contiguous() and k_cache.is_contiguous() and v_cache.is_contiguous()
    b, n_q, hd = q.shape
    n_kv = k_cache.shape[1]
    lib = load_library()
    cu = _cu_seqlens(seq_lens, q.device)
    nbytes = lib.swiftkv_tail_attention_scratch_bytes(b, n_q, hd, max(seq_lens))
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    out = torch.empty((b, n_q * hd), dtype=torch.float32, device=q.device)
    code = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[k_cache.dtype]
    with torch.cuda.device(q.device):
        _check(lib.swiftkv_tail_attention(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), out.data_ptr(), cu.data_ptr(),
                                          b, max(seq_lens), n_q, n_kv, hd, code, scratch.data_ptr(), nbytes,
                                          _stream_ptr(stream)))
    return out


def tail_attention_noalloc(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
                           cu_seqlens: torch.Tensor, max_seq_len: int, stream: Optional[torch.cuda.Stream] = None) -> None:
    """swiftkv_tail_attention_noalloc: like tail_attention, but the library keeps the split-KV partials in its own
    fixed device array, so neither this wrapper nor the library allocates anything: the caller passes the output
    tensor and the prompt offsets (device int32 [n_seqs+1]).  For callers whose memory is fully committed or who may
    not call the allocator where they run; problems needing more than 9 MiB of partials raise SwiftKVError(-2)."""
    b, n_q, hd = q.shape
    n_kv = k_cache.shape[1]
    code = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[k_cache.dtype]
    with torch.cuda.device(q.device):
        _check(load_library().swiftkv_tail_attention_noalloc(q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(),
                                                             out.data_ptr(), cu_seqlens.data_ptr(), b, max_seq_len, n_q, n_kv,
                                                             hd, code, _stream_ptr(stream)))


def quantize_rows_fp8(x: torch.Tensor, want_deq: bool = True, stream: Optional[torch.cuda.Stream] = None):
    """swiftkv_quantize_rows_fp8: x fp32 [rows, width] -> (codes uint8 [rows, width], scales fp32 [rows], deq fp32 or None)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 2
    rows, width = x.shape
    codes = torch.empty((rows, width), dtype=torch.uint8, device=x.device)
    scales = torch.empty(rows, dtype=torch.float32, device=x.device)
    deq = torch.empty_like(x) if want_deq else None
    with torch.cuda.device(x.device):
        _check(load_library().swiftkv_quantize_rows_fp8(x.data_ptr(), rows, width, codes.data_ptr(), scales.data_ptr(),
                                                        deq.data_ptr() if want_deq else None, _stream_ptr(stream)))
    return codes, scales, deq


def tail_attention_fp8(q: torch.Tensor, k_codes: torch.Tensor, v_codes: torch.Tensor, k_scale: torch.Tensor,
                       v_scale: torch.Tensor, seq_lens: Sequence[int], stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """swiftkv_tail_attention_fp8: q fp32 [n_seqs, n_q, hd]; codes uint8 [T, n_kv, hd]; scales fp32 [T] -> fp32 [n_seqs, n_q*hd]."""
    assert q.is_cuda and q.dtype == torch.float32 and q.is_contiguous()
    assert k_codes.dtype == torch.uint8 and v_codes.dtype == torch.uint8 and k_codes.is_contiguous() and v_codes.is_contiguous()
    assert k_scale.dtype == torch.float32 and v_scale.dtype == torch.float32
    b, n_q, hd = q.shape
    n_kv = k_codes.shape[1]
    lib = load_library()
    cu = _cu_seqlens(seq_lens, q.device)
    nbytes = lib.swiftkv_tail_attention_scratch_bytes(b, n_q, hd, max(seq_lens))
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    out = torch.empty((b, n_q * hd), dtype=torch.float32, device=q.device)
    with torch.cuda.device(q.device):
        _check(lib.swiftkv_tail_attention_fp8(q.data_ptr(), k_codes.data_ptr(), v_codes.data_ptr(), k_scale.data_ptr(),
                                              v_scale.data_ptr(), out.data_ptr(), cu.data_ptr(), b, max(seq_lens), n_q, n_kv, hd,
                                              scratch.data_ptr(), nbytes, _stream_ptr(stream)))
    return out
