"""ctypes binding of libmars.so: the same entry points as ``include/mars.h``, argument marshalling
only.  PyTorch appears here for device memory and streams; every step of the computation runs in
the library's CUDA kernels.  There is no fallback: if the shared library is missing the import of
any entry point raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int32, c_int64, c_size_t, c_uint64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmars.so")

MARS_OK = 0
STATUS_NAMES = {0: "MARS_OK", 1: "MARS_ERR_INVALID_ARG", 2: "MARS_ERR_UNSUPPORTED", 3: "MARS_ERR_CUDA",
                4: "MARS_ERR_KV_FULL", 5: "MARS_ERR_TIMEOUT", 6: "MARS_ERR_BAD_HANDLE", 7: "MARS_ERR_BAD_TOKEN",
                8: "MARS_ERR_TOO_LARGE"}
MARS_ERR_INVALID_ARG = 1
# bits of mars_set_prefill_lo_planes
MARS_LO_QKV, MARS_LO_OPROJ, MARS_LO_ROUTER, MARS_LO_GATE_UP, MARS_LO_DOWN = 1, 2, 4, 8, 16
MARS_LO_ALL, MARS_LO_DEFAULT = 31, 7
LAYER_FIELDS = ("attn_norm", "wqkv", "q_norm", "k_norm", "wo", "mlp_norm", "router", "w_gate_up", "w_down")


KERNEL_CLASSES = ("qkv", "attn", "attn_merge", "oproj", "router", "gate_up", "down", "combine", "lm_head", "sample",
                  "other")


class MarsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} "
                         f"({lib().mars_status_string(status).decode()}; cuda={lib().mars_last_cuda_error()})")


class mars_config_t(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "n_experts",
                                       "top_k", "expert_inter", "vocab", "qk_norm", "max_pos")] + \
               [("rope_theta", c_float), ("rms_eps", c_float)]


class mars_layer_t(ctypes.Structure):
    _fields_ = [(n, c_void_p) for n in LAYER_FIELDS]


class mars_weights_t(ctypes.Structure):
    _fields_ = [("embed", c_void_p), ("final_norm", c_void_p), ("lm_head", c_void_p), ("layers", POINTER(mars_layer_t))]


class mars_sampling_t(ctypes.Structure):
    _fields_ = [("temperature", c_float), ("top_p", c_float), ("greedy", c_int32), ("reserved", c_int32),
                ("seed", c_uint64), ("step", c_uint64)]


class mars_debug_t(ctypes.Structure):
    _fields_ = [("logits", c_void_p), ("hidden", c_void_p), ("router_w", c_void_p), ("router_idx", c_void_p),
                ("forced_idx", c_void_p), ("nucleus_mass", c_void_p), ("expert_off", c_void_p), ("slot_token", c_void_p)]


class mars_step_info_t(ctypes.Structure):
    _fields_ = [("kernel_launches", c_int64), ("attn_items", c_int64), ("kv_tokens_read", c_int64),
                ("kv_tokens_streamed", c_int64)]


# name -> (restype, argtypes); mirrors include/mars.h one to one
SIGNATURES = {
    "mars_workspace_bytes": (c_size_t, [POINTER(mars_config_t), c_int32, c_int32]),
    "mars_model_load": (c_int32, [POINTER(mars_config_t), POINTER(mars_weights_t), c_void_p, c_size_t, c_int32, c_int32,
                                  POINTER(c_void_p)]),
    "mars_model_free": (c_int32, [c_void_p]),
    "mars_kv_meta_bytes": (c_size_t, [c_int32, c_int32]),
    "mars_kv_alloc": (c_int32, [c_void_p, c_void_p, c_void_p, c_size_t, c_int32, c_int32, c_int32, c_void_p, c_size_t,
                                POINTER(c_void_p)]),
    "mars_kv_free": (c_int32, [c_void_p]),
    "mars_kv_num_pages": (c_int32, [c_void_p]),
    "mars_kv_free_pages": (c_int32, [c_void_p]),
    "mars_kv_seq_reserve": (c_int32, [c_void_p, c_int32, c_int32]),
    "mars_kv_seq_adopt": (c_int32, [c_void_p, c_int32, POINTER(c_int32), c_int32, c_int32]),
    "mars_kv_seq_set_len": (c_int32, [c_void_p, c_int32, c_int32]),
    "mars_kv_seq_release": (c_int32, [c_void_p, c_int32]),
    "mars_kv_seq_len": (c_int32, [c_void_p, c_int32]),
    "mars_kv_block_table": (c_int32, [c_void_p, c_int32, POINTER(c_int32), c_int32, POINTER(c_int32)]),
    "mars_kv_seq_image_bytes": (c_size_t, [c_void_p, c_int32]),
    "mars_kv_seq_export": (c_int32, [c_void_p, c_int32, c_void_p, c_size_t, c_void_p]),
    "mars_kv_seq_import": (c_int32, [c_void_p, c_int32, c_void_p, c_size_t, c_int32, c_void_p]),
    "mars_kv_seq_fork": (c_int32, [c_void_p, c_int32, c_int32, c_void_p]),
    "mars_kv_page_refs": (c_int32, [c_void_p, c_int32]),
    "mars_kv_share_reads": (c_int32, [c_void_p, c_int32]),
    "mars_decode_step": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_int32), c_void_p,
                                   POINTER(mars_sampling_t), c_void_p, c_void_p, POINTER(mars_debug_t)]),
    "mars_prefill_chunk": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_int32), POINTER(c_int32), c_void_p,
                                     POINTER(c_int32), POINTER(mars_sampling_t), c_void_p, c_void_p,
                                     POINTER(mars_debug_t)]),
    "mars_mixed_step": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_int32), c_void_p, c_int32,
                                  POINTER(c_int32), POINTER(c_int32), c_void_p, POINTER(c_int32), POINTER(mars_sampling_t),
                                  c_void_p, c_void_p, POINTER(mars_debug_t)]),
    "mars_score_chunk": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_int32), POINTER(c_int32), c_void_p,
                                   c_void_p, ctypes.c_float, c_void_p, POINTER(mars_debug_t)]),
    "mars_decode_step_host": (c_int32, [c_void_p, c_void_p, c_void_p, c_int32, POINTER(c_int32), c_void_p,
                                        POINTER(mars_sampling_t), c_void_p, c_void_p]),
    "mars_decode_step_static": (c_int32, [POINTER(mars_config_t), POINTER(mars_weights_t), c_void_p, c_void_p, c_size_t,
                                          c_int32, c_void_p, c_int32, POINTER(c_int32), c_void_p, c_int32, c_void_p,
                                          POINTER(mars_sampling_t), c_void_p, c_void_p]),
    "mars_poll_status": (c_int32, [c_void_p]),
    "mars_set_prefill_lo_planes": (c_int32, [c_void_p, c_int32]),
    "mars_debug_bounded_wait": (c_int32, [c_void_p, c_void_p, c_int32]),
    "mars_profile_enable": (c_int32, [c_void_p, c_int32]),
    "mars_profile_read": (c_int32, [c_void_p, POINTER(ctypes.c_double), POINTER(c_int64)]),
    "mars_last_step_info": (c_int32, [c_void_p, POINTER(mars_step_info_t)]),
    "mars_active_experts_device": (c_void_p, [c_void_p]),
    "mars_last_cuda_error": (c_int32, []),
    "mars_status_string": (c_char_p, [c_int32]),
    "mars_version": (c_char_p, []),
}

_lib = None


def lib() -> ctypes.CDLL:
    """Loads libmars.so; raises if it has not been built (python -m paper_2511_11373_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_11373_b200.build`")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(status: int, where: str):
    if status != MARS_OK:
        raise MarsError(status, where)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _i32_array(values):
    values = [int(v) for v in values]
    return (c_int32 * len(values))(*values), len(values)


def _stream_handle(stream) -> c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream)


def make_config(model: dict, max_pos: int) -> mars_config_t:
    return mars_config_t(model["n_layers"], model["hidden"], model["n_q_heads"], model["n_kv_heads"],
                         model["head_dim"], model["n_experts"], model["top_k"], model["expert_inter"], model["vocab"],
                         model.get("qk_norm", 0), max_pos, model.get("rope_theta", 1e6), model.get("rms_eps", 1e-6))


def make_sampling(greedy=True, temperature=1.0, top_p=1.0, seed=0, step=0) -> mars_sampling_t:
    return mars_sampling_t(float(temperature), float(top_p), int(bool(greedy)), 0, int(seed), int(step))


def make_debug(logits=None, hidden=None, router_w=None, router_idx=None, forced_idx=None, nucleus_mass=None,
               expert_off=None, slot_token=None):
    taps = (logits, hidden, router_w, router_idx, forced_idx, nucleus_mass, expert_off, slot_token)
    d = mars_debug_t(*[t.data_ptr() if t is not None else None for t in taps])
    d._keep = taps
    return d


class Model:
    """mars_model_load / mars_model_free.  `weights` is the nested dict of CUDA bf16 tensors produced by
    ``workloads.make_weights``; the tensors are borrowed, not copied, and are kept alive here."""

    def __init__(self, model: dict, weights: dict, max_decode_seqs: int, max_prefill_tokens: int = 0,
                 max_pos: int = 4096):
        self.shape = dict(model)
        self.cfg = make_config(model, max_pos)
        self.weights = weights
        self.max_decode_seqs, self.max_prefill_tokens = max_decode_seqs, max_prefill_tokens
        nbytes = lib().mars_workspace_bytes(byref(self.cfg), max_decode_seqs, max_prefill_tokens)
        if nbytes == 0:
            raise MarsError(2, "mars_workspace_bytes")
        dev = weights["embed"].device
        self.device = dev
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        layers = (mars_layer_t * len(weights["layers"]))()
        for i, layer in enumerate(weights["layers"]):
            for f in LAYER_FIELDS:
                t = layer[f]
                assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
                setattr(layers[i], f, t.data_ptr())
        w = mars_weights_t(weights["embed"].data_ptr(), weights["final_norm"].data_ptr(), weights["lm_head"].data_ptr(),
                           layers)
        self._layers = layers
        handle = c_void_p()
        with torch.cuda.device(dev):
            _check(lib().mars_model_load(byref(self.cfg), byref(w), _ptr(self.workspace), nbytes, max_decode_seqs,
                                         max_prefill_tokens, byref(handle)), "mars_model_load")
        self.handle = handle

    def poll_status(self) -> int:
        return lib().mars_poll_status(self.handle)

    def bounded_wait_selftest(self, arrive: bool, stream=None) -> int:
        """Launches the library's bounded-wait self-test (see mars_debug_bounded_wait); returns the status code."""
        with torch.cuda.device(self.device):
            return lib().mars_debug_bounded_wait(self.handle, _stream_handle(stream), 1 if arrive else 0)

    def set_prefill_lo_planes(self, mask: int):
        """Bit per contraction class of large calls (QKV 1, output projection 2, router 4, gate/up 8, down 16):
        set = (hi, lo) activations, clear = hi plane only."""
        _check(lib().mars_set_prefill_lo_planes(self.handle, int(mask)), "mars_set_prefill_lo_planes")

    def last_step_info(self) -> dict:
        info = mars_step_info_t()
        _check(lib().mars_last_step_info(self.handle, byref(info)), "mars_last_step_info")
        return dict(kernel_launches=info.kernel_launches, attn_items=info.attn_items,
                    kv_tokens_read=info.kv_tokens_read, kv_tokens_streamed=info.kv_tokens_streamed)

    def profile_enable(self, on: bool = True):
        _check(lib().mars_profile_enable(self.handle, int(on)), "mars_profile_enable")

    def profile_read(self) -> dict:
        """{class name: (milliseconds, launches)} accumulated since the last read."""
        ms = (ctypes.c_double * len(KERNEL_CLASSES))()
        n = (c_int64 * len(KERNEL_CLASSES))()
        _check(lib().mars_profile_read(self.handle, ms, n), "mars_profile_read")
        return {name: (ms[i], n[i]) for i, name in enumerate(KERNEL_CLASSES)}

    def active_experts(self) -> torch.Tensor:
        """Distinct experts selected per layer in the last step (copied to the host; synchronises)."""
        p = lib().mars_active_experts_device(self.handle)
        out = torch.empty(self.shape["n_layers"], dtype=torch.int32, device=self.device)
        n = self.shape["n_layers"] * 4
        torch.cuda.synchronize(self.device)
        # device-to-device view of the library's counter array, through the workspace tensor
        off = p - self.workspace.data_ptr()
        out.copy_(self.workspace[off:off + n].view(torch.int32))
        return out.cpu()

    def close(self):
        if getattr(self, "handle", None):
            lib().mars_model_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class KvCache:
    """mars_kv_alloc / mars_kv_free and the per-sequence calls.  The pools are caller tensors of shape
    [n_layers, n_pages, n_kv_heads, page_size, head_dim] (bf16)."""

    def __init__(self, model: Model, k_pool: torch.Tensor, v_pool: torch.Tensor, page_size: int, max_seqs: int,
                 max_pages_per_seq: int):
        assert k_pool.is_cuda and k_pool.dtype == torch.bfloat16 and k_pool.is_contiguous() and k_pool.shape == v_pool.shape
        self.model, self.k_pool, self.v_pool = model, k_pool, v_pool
        self.page_size, self.max_seqs, self.max_pages_per_seq = page_size, max_seqs, max_pages_per_seq
        nmeta = lib().mars_kv_meta_bytes(max_seqs, max_pages_per_seq)
        self.meta = torch.empty(nmeta, dtype=torch.uint8, device=k_pool.device)
        handle = c_void_p()
        with torch.cuda.device(k_pool.device):
            _check(lib().mars_kv_alloc(model.handle, _ptr(k_pool), _ptr(v_pool), k_pool.numel() * 2, page_size, max_seqs,
                                       max_pages_per_seq, _ptr(self.meta), nmeta, byref(handle)), "mars_kv_alloc")
        self.handle = handle

    @property
    def num_pages(self) -> int:
        return lib().mars_kv_num_pages(self.handle)

    @property
    def free_pages(self) -> int:
        return lib().mars_kv_free_pages(self.handle)

    def seq_reserve(self, seq: int, n_tokens_total: int):
        _check(lib().mars_kv_seq_reserve(self.handle, seq, n_tokens_total), "mars_kv_seq_reserve")

    def seq_adopt(self, seq: int, pages, ctx_len: int):
        arr, n = _i32_array(pages)
        _check(lib().mars_kv_seq_adopt(self.handle, seq, arr, n, ctx_len), "mars_kv_seq_adopt")

    def seq_set_len(self, seq: int, ctx_len: int):
        _check(lib().mars_kv_seq_set_len(self.handle, seq, ctx_len), "mars_kv_seq_set_len")

    def seq_release(self, seq: int):
        _check(lib().mars_kv_seq_release(self.handle, seq), "mars_kv_seq_release")

    def seq_len(self, seq: int) -> int:
        return lib().mars_kv_seq_len(self.handle, seq)

    def block_table(self, seq: int):
        arr = (c_int32 * self.max_pages_per_seq)()
        n = c_int32()
        _check(lib().mars_kv_block_table(self.handle, seq, arr, self.max_pages_per_seq, byref(n)), "mars_kv_block_table")
        return list(arr[: n.value])

    def seq_image_bytes(self, n_tokens: int) -> int:
        return lib().mars_kv_seq_image_bytes(self.handle, n_tokens)

    def seq_export(self, seq: int, image: torch.Tensor, stream=None) -> int:
        """`image`: uint8 tensor on the device or in pinned host memory.  Returns the status code."""
        with torch.cuda.device(self.k_pool.device):
            return lib().mars_kv_seq_export(self.handle, seq, image.data_ptr(), image.numel() * image.element_size(),
                                            _stream_handle(stream))

    def seq_import(self, seq: int, image: torch.Tensor, n_tokens: int, stream=None) -> int:
        with torch.cuda.device(self.k_pool.device):
            return lib().mars_kv_seq_import(self.handle, seq, image.data_ptr(), image.numel() * image.element_size(),
                                            n_tokens, _stream_handle(stream))

    def seq_fork(self, src: int, dst: int, stream=None) -> int:
        with torch.cuda.device(self.k_pool.device):
            return lib().mars_kv_seq_fork(self.handle, src, dst, _stream_handle(stream))

    def page_refs(self, page: int) -> int:
        return lib().mars_kv_page_refs(self.handle, page)

    def share_reads(self, enable: bool) -> None:
        _check(lib().mars_kv_share_reads(self.handle, 1 if enable else 0), "mars_kv_share_reads")

    def close(self):
        if getattr(self, "handle", None):
            lib().mars_kv_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def mars_decode_step(model: Model, kv: KvCache, seq_ids, in_tokens: torch.Tensor, sampling: mars_sampling_t,
                     out_tokens: torch.Tensor, out_logprobs: torch.Tensor, debug: mars_debug_t | None = None,
                     stream=None) -> int:
    """Returns the status code (0 = ok) without raising, so that error paths can be tested."""
    arr, n = _i32_array(seq_ids)
    return lib().mars_decode_step(model.handle, kv.handle, _stream_handle(stream), n, arr, _ptr(in_tokens),
                                  byref(sampling), _ptr(out_tokens), _ptr(out_logprobs),
                                  byref(debug) if debug is not None else None)


def mars_prefill_chunk(model: Model, kv: KvCache, seq_ids, chunk_lens, tokens: torch.Tensor, emit_last,
                       sampling: mars_sampling_t, out_tokens, out_logprobs, debug: mars_debug_t | None = None,
                       stream=None) -> int:
    ids, n = _i32_array(seq_ids)
    lens, _ = _i32_array(chunk_lens)
    emit, _ = _i32_array(emit_last) if emit_last is not None else (None, 0)
    return lib().mars_prefill_chunk(model.handle, kv.handle, _stream_handle(stream), n, ids, lens, _ptr(tokens), emit,
                                    byref(sampling), _ptr(out_tokens), _ptr(out_logprobs),
                                    byref(debug) if debug is not None else None)


def mars_mixed_step(model: Model, kv: KvCache, seq_ids, in_tokens: torch.Tensor, req_ids, chunk_lens,
                    chunk_tokens: torch.Tensor, emit_last, sampling: mars_sampling_t, out_tokens: torch.Tensor,
                    out_logprobs: torch.Tensor, debug: mars_debug_t | None = None, stream=None) -> int:
    """Decode rows and prompt chunks in one pass; outputs: decode rows first, then the emitting requests."""
    ids, n = _i32_array(seq_ids)
    rids, nr = _i32_array(req_ids)
    lens, _ = _i32_array(chunk_lens)
    emit, _ = _i32_array(emit_last) if emit_last is not None else (None, 0)
    return lib().mars_mixed_step(model.handle, kv.handle, _stream_handle(stream), n, ids, _ptr(in_tokens), nr, rids, lens,
                                 _ptr(chunk_tokens), emit, byref(sampling), _ptr(out_tokens), _ptr(out_logprobs),
                                 byref(debug) if debug is not None else None)


def mars_score_chunk(model: Model, kv: KvCache, seq_ids, chunk_lens, tokens: torch.Tensor, targets: torch.Tensor,
                     temperature: float, out_logprobs: torch.Tensor, debug: mars_debug_t | None = None, stream=None) -> int:
    """Teacher-forced log-probs of `targets` (one per token row, < 0 = none); returns the status code."""
    ids, n = _i32_array(seq_ids)
    lens, _ = _i32_array(chunk_lens)
    return lib().mars_score_chunk(model.handle, kv.handle, _stream_handle(stream), n, ids, lens, _ptr(tokens),
                                  _ptr(targets), float(temperature), _ptr(out_logprobs),
                                  byref(debug) if debug is not None else None)


def mars_decode_step_host(model: Model, kv: KvCache, seq_ids, in_tokens_host: torch.Tensor, sampling: mars_sampling_t,
                          out_tokens_host: torch.Tensor, out_logprobs_host: torch.Tensor, stream=None) -> int:
    """Host-buffer variant: CPU int32 / fp32 tensors in and out, copies included, synchronous."""
    arr, n = _i32_array(seq_ids)
    assert not in_tokens_host.is_cuda and not out_tokens_host.is_cuda and not out_logprobs_host.is_cuda
    return lib().mars_decode_step_host(model.handle, kv.handle, _stream_handle(stream), n, arr, _ptr(in_tokens_host),
                                       byref(sampling), _ptr(out_tokens_host), _ptr(out_logprobs_host))


def mars_decode_step_static(model_shape: dict, weights: dict, max_pos: int, k_pool: torch.Tensor, v_pool: torch.Tensor,
                            page_size: int, block_table: torch.Tensor, ctx_lens, in_tokens: torch.Tensor,
                            sampling: mars_sampling_t, out_tokens: torch.Tensor, out_logprobs: torch.Tensor,
                            stream=None) -> int:
    """Decode step that needs no handle and no workspace (for callers that cannot allocate device
    memory): its intermediates live in a fixed array inside the library.  `block_table` is a CUDA int32
    tensor [n_seqs, max_pages_per_seq]; `ctx_lens` a host list.  Returns the status code."""
    cfg = make_config(model_shape, max_pos)
    layers = (mars_layer_t * len(weights["layers"]))()
    for i, layer in enumerate(weights["layers"]):
        for f in LAYER_FIELDS:
            setattr(layers[i], f, layer[f].data_ptr())
    w = mars_weights_t(weights["embed"].data_ptr(), weights["final_norm"].data_ptr(), weights["lm_head"].data_ptr(), layers)
    lens, n = _i32_array(ctx_lens)
    assert block_table.is_cuda and block_table.dtype == torch.int32 and block_table.is_contiguous()
    with torch.cuda.device(k_pool.device):
        return lib().mars_decode_step_static(byref(cfg), byref(w), _ptr(k_pool), _ptr(v_pool), k_pool.numel() * 2,
                                             page_size, _ptr(block_table), block_table.shape[1], lens,
                                             _stream_handle(stream), n, _ptr(in_tokens), byref(sampling),
                                             _ptr(out_tokens), _ptr(out_logprobs))
