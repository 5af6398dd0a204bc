"""ctypes binding of include/rpo.h: same names, argument marshalling only.

Device buffers are torch CUDA tensors (their data pointers are passed through); every
step of the path runs inside the library's kernels.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

EXPORTED_SYMBOLS = [
    "rpo_strerror", "rpo_shape_preset", "rpo_create", "rpo_destroy", "rpo_init_weights", "rpo_read_tensor",
    "rpo_write_tensor", "rpo_prefill_prefix", "rpo_decode_suffix", "rpo_decode_wave", "rpo_token_logprobs", "rpo_release_groups",
    "rpo_policy_objective", "rpo_rollout_host", "rpo_sample_rows", "rpo_sample_rows_noalloc", "rpo_gemm", "rpo_gemm_bench", "rpo_device_status", "rpo_debug_tap", "rpo_counters", "rpo_set_option", "rpo_profile_read",
]


class RpoError(RuntimeError):
    def __init__(self, code, what):
        super().__init__(f"{what}: {code} ({load_library().rpo_strerror(code).decode()})")
        self.code = code


class Shape(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("rope_base", C.c_float),
                ("rms_eps", C.c_float), ("dtype", C.c_int32), ("kv_block_tokens", C.c_int32)]


class Limits(C.Structure):
    _fields_ = [("kv_pool_blocks", C.c_int64), ("max_groups", C.c_int32), ("max_seqs", C.c_int32),
                ("max_chunk_tokens", C.c_int32), ("max_positions", C.c_int32)]


class Sampler(C.Structure):
    _fields_ = [("temperature", C.c_float), ("top_p", C.c_float), ("greedy", C.c_int32), ("eos_id", C.c_int32),
                ("seed", C.c_uint64)]

    def __init__(self, temperature=1.0, top_p=1.0, greedy=False, eos_id=-1, seed=0):
        super().__init__(float(temperature), float(top_p), int(bool(greedy)), int(eos_id), int(seed))


class ObjectiveCfg(C.Structure):
    _fields_ = [("clip_eps", C.c_float), ("beta", C.c_float), ("alpha", C.c_float), ("reward_min", C.c_float),
                ("reward_max", C.c_float), ("length_shaping", C.c_int32)]

    def __init__(self, clip_eps=0.2, beta=0.0, alpha=0.01, reward_min=0.5, reward_max=1.0, length_shaping=True):
        super().__init__(float(clip_eps), float(beta), float(alpha), float(reward_min), float(reward_max), int(bool(length_shaping)))


class Group(C.Structure):
    _fields_ = [("group_id", C.c_int32), ("prefix_len", C.c_int32), ("slot", C.c_int32), ("n_blocks", C.c_int32)]


def load_library(path=None):
    """Load librpo.so (building it first if it is missing) and declare the prototypes."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    path = path or os.path.join(_HERE, "librpo.so")
    if not os.path.exists(path):
        from . import build as _build
        _build.build()
    lib = C.CDLL(path)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.rpo_strerror.restype = C.c_char_p; lib.rpo_strerror.argtypes = [C.c_int]
    lib.rpo_shape_preset.argtypes = [C.c_char_p, C.POINTER(Shape)]
    lib.rpo_create.argtypes = [C.POINTER(vp), C.POINTER(Shape), C.POINTER(Limits), vp]
    lib.rpo_destroy.argtypes = [vp]
    lib.rpo_init_weights.argtypes = [vp, C.c_uint64, f32]
    lib.rpo_read_tensor.argtypes = [vp, C.c_char_p, vp, C.c_size_t]
    lib.rpo_write_tensor.argtypes = [vp, C.c_char_p, vp, C.c_size_t]
    lib.rpo_prefill_prefix.argtypes = [vp, i32, vp, vp, vp, C.POINTER(Group)]
    lib.rpo_decode_suffix.argtypes = [vp, i32, C.POINTER(Group), i32, i32, C.POINTER(Sampler), vp, vp, vp, vp, vp]
    lib.rpo_decode_wave.argtypes = [vp, i32, C.POINTER(Group), i32, i32, i32, C.POINTER(Sampler), vp, vp, vp, vp]
    lib.rpo_token_logprobs.argtypes = [vp, i32, C.POINTER(Group), i32, i32, vp, vp, f32, vp, vp]
    lib.rpo_policy_objective.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, C.POINTER(ObjectiveCfg), vp, vp, vp, vp, vp]
    lib.rpo_release_groups.argtypes = [vp, i32, C.POINTER(Group)]
    lib.rpo_rollout_host.argtypes = [vp, i32, vp, vp, vp, i32, i32, C.POINTER(Sampler), vp, vp, vp, i32, vp]
    lib.rpo_sample_rows.argtypes = [vp, i32, i32, vp, C.POINTER(Sampler), vp, i32, vp, vp]
    lib.rpo_sample_rows_noalloc.argtypes = [i32, i32, vp, C.POINTER(Sampler), vp, i32, vp, vp, vp]
    lib.rpo_gemm.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp]
    lib.rpo_gemm_bench.argtypes = [vp, i32, i32, i32, vp, C.POINTER(vp), i32, i32, C.POINTER(f32)]
    lib.rpo_device_status.argtypes = [vp, C.POINTER(i32)]
    lib.rpo_debug_tap.argtypes = [vp, vp, i64, C.POINTER(i64)]
    lib.rpo_counters.argtypes = [vp, C.POINTER(i64), C.POINTER(i64)]
    lib.rpo_set_option.argtypes = [vp, C.c_char_p, i32]
    lib.rpo_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64), i32]
    for name in EXPORTED_SYMBOLS:
        if name != "rpo_strerror":
            getattr(lib, name).restype = C.c_int
    if path == os.path.join(_HERE, "librpo.so"):
        _LIB = lib
    return lib


def shape_preset(name, **overrides):
    s = Shape()
    rc = load_library().rpo_shape_preset(name.encode(), C.byref(s))
    if rc != 0:
        raise RpoError(rc, f"rpo_shape_preset({name})")
    for k, v in overrides.items():
        setattr(s, k, v)
    return s


def shape_from_dict(d):
    s = Shape()
    for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab"):
        setattr(s, k, int(d[k]))
    s.rope_base = float(d.get("rope_base", 10000.0)); s.rms_eps = float(d.get("rms_eps", 1e-6))
    s.dtype = 1 if d.get("dtype", "fp32") == "bf16" else 0
    s.kv_block_tokens = 16
    return s


def _ptr(t):
    """Device/host pointer of a torch tensor or numpy array (None -> NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous()
    return t.data_ptr()


def _check(rc, what):
    if rc != 0:
        raise RpoError(rc, what)


def sample_rows_noalloc(d_logits, sampler, d_seq_ids, step, d_tokens_out, d_logprobs_out=None, stream=None):
    """rpo_sample_rows_noalloc: the sampler on caller-supplied logits [n_rows, vocab] without a context
    and without any allocation (its scratch is a fixed 16 MiB array inside the library, so
    n_rows * vocab is limited to 4 Mi words).  `stream` is a torch.cuda.Stream or None."""
    n, v = d_logits.shape
    stream_ptr = None if stream is None else C.c_void_p(stream.cuda_stream)
    _check(load_library().rpo_sample_rows_noalloc(n, v, _ptr(d_logits), C.byref(sampler), _ptr(d_seq_ids), int(step),
                                                  _ptr(d_tokens_out), _ptr(d_logprobs_out), stream_ptr),
           "rpo_sample_rows_noalloc")


class Context:
    """Owns one rpo_ctx.  Methods mirror the C calls one to one."""

    def __init__(self, shape, kv_pool_blocks, max_groups, max_seqs, max_chunk_tokens, max_positions, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2601_19404_b200 needs a CUDA device: the library has no CPU path")
        self.lib = load_library()
        self.shape = shape if isinstance(shape, Shape) else shape_from_dict(shape)
        self.limits = Limits(int(kv_pool_blocks), int(max_groups), int(max_seqs), int(max_chunk_tokens), int(max_positions))
        self.handle = C.c_void_p()
        stream_ptr = None if stream is None else C.c_void_p(stream.cuda_stream)
        _check(self.lib.rpo_create(C.byref(self.handle), C.byref(self.shape), C.byref(self.limits), stream_ptr), "rpo_create")

    def close(self):
        h = getattr(self, "handle", None)
        if h is not None and h.value:
            self.lib.rpo_destroy(h)
            h.value = None

    __del__ = close

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    @property
    def storage_dtype(self):
        return np.uint16 if self.shape.dtype == 1 else np.float32

    def init_weights(self, seed=0, std=0.02):
        _check(self.lib.rpo_init_weights(self.handle, int(seed), float(std)), "rpo_init_weights")

    def tensor_shape(self, name):
        s = self.shape
        qo, kvo = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
        leaf = name.split(".")[-1]
        table = {"embed": (s.vocab, s.d_model), "lm_head": (s.vocab, s.d_model), "gf": (s.d_model,),
                 "wq": (qo, s.d_model), "wk": (kvo, s.d_model), "wv": (kvo, s.d_model), "wo": (s.d_model, qo),
                 "wg": (s.d_ffn, s.d_model), "wu": (s.d_ffn, s.d_model), "wd": (s.d_model, s.d_ffn),
                 "g1": (s.d_model,), "g2": (s.d_model,)}
        return table[leaf]

    def read_tensor(self, name):
        gain = name.split(".")[-1] in ("gf", "g1", "g2")
        out = np.empty(self.tensor_shape(name), dtype=np.float32 if gain else self.storage_dtype)
        _check(self.lib.rpo_read_tensor(self.handle, name.encode(), out.ctypes.data, out.nbytes), f"rpo_read_tensor({name})")
        return out

    def write_tensor(self, name, array):
        gain = name.split(".")[-1] in ("gf", "g1", "g2")
        a = np.ascontiguousarray(array, dtype=np.float32 if gain else self.storage_dtype)
        assert a.shape == tuple(self.tensor_shape(name))
        _check(self.lib.rpo_write_tensor(self.handle, name.encode(), a.ctypes.data, a.nbytes), f"rpo_write_tensor({name})")

    def prefill_prefix(self, d_tokens, h_offsets, group_ids=None):
        n = len(h_offsets) - 1
        off = np.ascontiguousarray(h_offsets, dtype=np.int32)
        ids = None if group_ids is None else np.ascontiguousarray(group_ids, dtype=np.int32)
        groups = (Group * n)()
        _check(self.lib.rpo_prefill_prefix(self.handle, n, _ptr(d_tokens), off.ctypes.data,
                                           None if ids is None else ids.ctypes.data, groups), "rpo_prefill_prefix")
        return groups

    def decode_suffix(self, groups, G, max_new, sampler, d_tokens_out, d_lens_out, d_logprobs_out=None,
                      d_forced_tokens=None, d_logits_dbg=None):
        _check(self.lib.rpo_decode_suffix(self.handle, len(groups), groups, int(G), int(max_new), C.byref(sampler),
                                          _ptr(d_forced_tokens), _ptr(d_tokens_out), _ptr(d_lens_out),
                                          _ptr(d_logprobs_out), _ptr(d_logits_dbg)), "rpo_decode_suffix")

    def decode_wave(self, groups, G, max_new, max_total, sampler, d_tokens_out, d_lens_out, d_logprobs_out=None,
                    d_forced_tokens=None):
        _check(self.lib.rpo_decode_wave(self.handle, len(groups), groups, int(G), int(max_new), int(max_total),
                                        C.byref(sampler), _ptr(d_forced_tokens), _ptr(d_tokens_out), _ptr(d_lens_out),
                                        _ptr(d_logprobs_out)), "rpo_decode_wave")

    def token_logprobs(self, groups, G, max_new, d_tokens, d_lens, d_logprobs_out, inv_temperature=1.0, d_logits_dbg=None):
        _check(self.lib.rpo_token_logprobs(self.handle, len(groups), groups, int(G), int(max_new), _ptr(d_tokens),
                                           _ptr(d_lens), float(inv_temperature), _ptr(d_logprobs_out),
                                           _ptr(d_logits_dbg)), "rpo_token_logprobs")

    def policy_objective(self, n_groups, G, max_new, d_logp_new, d_logp_old, d_lens, d_raw_rewards, cfg, d_rewards_out,
                         d_advantages_out, d_group_objective_out, d_objective_out, d_logp_ref=None, d_resp_lens=None,
                         d_token_loss_out=None):
        _check(self.lib.rpo_policy_objective(self.handle, int(n_groups), int(G), int(max_new), _ptr(d_logp_new), _ptr(d_logp_old),
                                             _ptr(d_logp_ref), _ptr(d_lens), _ptr(d_resp_lens), _ptr(d_raw_rewards), C.byref(cfg),
                                             _ptr(d_rewards_out), _ptr(d_advantages_out), _ptr(d_token_loss_out),
                                             _ptr(d_group_objective_out), _ptr(d_objective_out)), "rpo_policy_objective")

    def release_groups(self, groups):
        _check(self.lib.rpo_release_groups(self.handle, len(groups), groups), "rpo_release_groups")

    def rollout_host(self, h_tokens, h_offsets, G, max_new, sampler, h_tokens_out, h_lens_out, h_logprobs_out=None,
                     h_policy_logprobs_out=None, group_ids=None):
        n = len(h_offsets) - 1
        off = np.ascontiguousarray(h_offsets, dtype=np.int32)
        ids = None if group_ids is None else np.ascontiguousarray(group_ids, dtype=np.int32)
        _check(self.lib.rpo_rollout_host(self.handle, n, _ptr(h_tokens), off.ctypes.data,
                                         None if ids is None else ids.ctypes.data, int(G), int(max_new),
                                         C.byref(sampler), _ptr(h_tokens_out), _ptr(h_lens_out), _ptr(h_logprobs_out),
                                         int(h_policy_logprobs_out is not None), _ptr(h_policy_logprobs_out)),
               "rpo_rollout_host")

    def sample_rows(self, d_logits, sampler, d_seq_ids, step, d_tokens_out, d_logprobs_out=None):
        n, v = d_logits.shape
        _check(self.lib.rpo_sample_rows(self.handle, n, v, _ptr(d_logits), C.byref(sampler), _ptr(d_seq_ids), int(step),
                                        _ptr(d_tokens_out), _ptr(d_logprobs_out)), "rpo_sample_rows")

    def gemm(self, d_A, d_W, d_C, impl=0):
        M, K = d_A.shape
        N = d_W.shape[0]
        _check(self.lib.rpo_gemm(self.handle, int(impl), M, N, K, _ptr(d_A), _ptr(d_W), _ptr(d_C)), "rpo_gemm")

    def gemm_bench(self, d_A, d_W_list, iters):
        """Mean device milliseconds per launch of the tensor-core GEMM A W^T, cycling through d_W_list."""
        M, K = d_A.shape
        N = d_W_list[0].shape[0]
        ptrs = (C.c_void_p * len(d_W_list))(*[w.data_ptr() for w in d_W_list])
        ms = C.c_float()
        _check(self.lib.rpo_gemm_bench(self.handle, M, N, K, _ptr(d_A), ptrs, len(d_W_list), int(iters), C.byref(ms)),
               "rpo_gemm_bench")
        return ms.value

    def device_status(self, raise_on_timeout=True):
        """The device status word (cleared by the read).  An expired device-side wait (bit 0) raises
        RpoError(RPO_ERR_DEVICE_TIMEOUT) unless raise_on_timeout is False."""
        v = C.c_int32()
        rc = self.lib.rpo_device_status(self.handle, C.byref(v))
        if rc != 0 and (raise_on_timeout or rc != -5):
            raise RpoError(rc, "rpo_device_status")
        return v.value

    def debug_tap(self, d_buf):
        """Set (tensor) or clear (None) the residual-stream tap; returns the floats written so far."""
        used = C.c_int64()
        _check(self.lib.rpo_debug_tap(self.handle, _ptr(d_buf), 0 if d_buf is None else d_buf.numel(), C.byref(used)),
               "rpo_debug_tap")
        return used.value

    def counters(self):
        a, b = C.c_int64(), C.c_int64()
        _check(self.lib.rpo_counters(self.handle, C.byref(a), C.byref(b)), "rpo_counters")
        return a.value, b.value

    def set_option(self, name, value):
        _check(self.lib.rpo_set_option(self.handle, name.encode(), int(value)), f"rpo_set_option({name})")

    PHASES = ("prefill", "decode", "logprobs")
    CLASSES = ("other", "gemm", "attention", "sampler", "rmsnorm", "rope_kv")

    def profile_read(self):
        """{phase: {class: (total_ms, launches)}} since the last read (needs option profile=1)."""
        n = len(self.PHASES) * len(self.CLASSES)
        ms = (C.c_double * n)(); cnt = (C.c_int64 * n)()
        _check(self.lib.rpo_profile_read(self.handle, ms, cnt, n), "rpo_profile_read")
        return {p: {k: (ms[i * len(self.CLASSES) + j], cnt[i * len(self.CLASSES) + j])
                    for j, k in enumerate(self.CLASSES)} for i, p in enumerate(self.PHASES)}
