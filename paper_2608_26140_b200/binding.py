"""Thin ctypes binding of the C-ABI library (``include/acache.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are ``torch`` CUDA tensors (used for device memory and the
current stream); there is no CPU fallback -- loading fails loudly if the
library has not been built (``python -m paper_2608_26140_b200.build``).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libacache.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
FLAG_BAD_INDEX, FLAG_WAIT_EXPIRED = 0x1, 0x2
F_SCORE, F_SELECT, F_ACCUMULATE, F_SCORE_NORM_FULL, F_NO_RECOMPUTE, F_DROP_NON_ANCHOR = 0x1, 0x2, 0x4, 0x8, 0x10, 0x20

EXPORTS = ["acache_create", "acache_workspace_bytes", "acache_set_workspace", "acache_destroy",
           "acache_last_error", "acache_poll_status", "acache_launch_count", "acache_score_anchors",
           "acache_k_from_ratio", "acache_select_topk", "acache_recompute_anchors", "acache_scatter_kv",
           "acache_layer_step", "acache_layer_step_host", "acache_stage_timing", "acache_read_stage_times",
           "acache_score_anchors_static", "acache_predict_commit", "acache_denoise_step", "acache_probe_select",
           "acache_commit_update", "acache_generate_block", "acache_denoise_step_shared", "acache_recompute_rows_shared",
           "acache_decode_step_shared", "acache_generate_block_shared", "acache_layer_step_shared",
           "acache_host_x_in_place", "acache_score_kv_deviation", "acache_debug_expire_next_wait"]

STAGES = ["mask_q", "score", "topk", "gather_norm", "qkv", "attention", "oproj", "mlp_norm", "gate_up", "down"]


class ModelDesc(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("rms_eps", C.c_float),
                ("qkv_bias", C.c_int32), ("max_batch", C.c_int32), ("max_ctx", C.c_int32),
                ("max_affix", C.c_int32), ("max_rows", C.c_int32), ("max_masked", C.c_int32),
                ("max_vocab", C.c_int32), ("max_block", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm_g", "wq", "wk", "wv", "bq", "bk", "bv", "wo",
                                          "mlp_norm_g", "w_gate", "w_up", "w_down")]


class KV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("batch_stride", C.c_int64), ("ctx_capacity", C.c_int32)]


class Request(C.Structure):
    _fields_ = [("batch", C.c_int32), ("ctx_len", C.c_int32), ("affix_start", C.c_int32),
                ("affix_len", C.c_int32), ("masked_pos", C.c_void_p), ("n_masked", C.c_int32),
                ("extra_rows", C.c_void_p), ("n_extra", C.c_int32), ("rope_cos", C.c_void_p),
                ("rope_sin", C.c_void_p), ("token_ids", C.c_void_p), ("n_embed", C.c_int32)]


class AcacheError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"acache status {status}: {msg}")
        self.status = status


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads libacache.so (once) and declares the prototypes."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} is missing: build it with `python -m paper_2608_26140_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(p)
    vp, i32, u32, i64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_int64
    lib.acache_create.argtypes = [C.POINTER(ModelDesc), C.POINTER(vp)]
    lib.acache_create.restype = C.c_int
    lib.acache_workspace_bytes.argtypes = [vp]
    lib.acache_workspace_bytes.restype = C.c_size_t
    lib.acache_set_workspace.argtypes = [vp, vp, C.c_size_t, vp]
    lib.acache_set_workspace.restype = C.c_int
    lib.acache_destroy.argtypes = [vp]
    lib.acache_destroy.restype = None
    lib.acache_last_error.argtypes = [vp]
    lib.acache_last_error.restype = C.c_char_p
    lib.acache_poll_status.argtypes = [vp, vp, C.POINTER(u32)]
    lib.acache_poll_status.restype = C.c_int
    lib.acache_debug_expire_next_wait.argtypes = [vp]
    lib.acache_debug_expire_next_wait.restype = C.c_int
    lib.acache_launch_count.argtypes = [vp]
    lib.acache_launch_count.restype = C.c_uint64
    lib.acache_score_anchors.argtypes = [vp, C.POINTER(Request), vp, C.POINTER(KV), vp, C.c_int, C.c_int, vp]
    lib.acache_score_anchors.restype = C.c_int
    lib.acache_score_kv_deviation.argtypes = [vp, C.POINTER(Request), C.POINTER(KV), C.POINTER(KV), vp, C.c_int, vp]
    lib.acache_score_kv_deviation.restype = C.c_int
    lib.acache_k_from_ratio.argtypes = [i32, C.c_double]
    lib.acache_k_from_ratio.restype = i32
    lib.acache_select_topk.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    lib.acache_select_topk.restype = C.c_int
    lib.acache_recompute_anchors.argtypes = [vp, C.POINTER(LayerWeights), C.POINTER(Request), C.POINTER(KV),
                                             vp, C.c_int, vp, i32, vp, vp, vp, vp]
    lib.acache_recompute_anchors.restype = C.c_int
    lib.acache_scatter_kv.argtypes = [vp, C.POINTER(Request), C.POINTER(KV), vp, i32, vp, vp, vp]
    lib.acache_scatter_kv.restype = C.c_int
    lib.acache_layer_step.argtypes = [vp, C.POINTER(LayerWeights), C.POINTER(Request), C.POINTER(KV), vp, C.c_int,
                                      C.c_double, u32, vp, vp, vp, vp]
    lib.acache_layer_step.restype = C.c_int
    lib.acache_layer_step_host.argtypes = [vp, C.POINTER(LayerWeights), C.POINTER(Request), C.POINTER(KV), vp,
                                           C.c_double, u32, vp, vp, vp, vp]
    lib.acache_layer_step_host.restype = C.c_int
    lib.acache_host_x_in_place.argtypes = [vp]
    lib.acache_host_x_in_place.restype = C.c_int32
    lib.acache_score_anchors_static.argtypes = [C.POINTER(ModelDesc), C.POINTER(Request), vp, C.POINTER(KV), vp,
                                                C.c_int, C.c_int, vp]
    lib.acache_score_anchors_static.restype = C.c_int
    lib.acache_predict_commit.argtypes = [vp, vp, i32, vp, i32, i32, vp, vp, i32, C.c_float, vp, vp, vp, vp]
    lib.acache_predict_commit.restype = C.c_int
    lib.acache_denoise_step.argtypes = [vp, i32, C.POINTER(LayerWeights), C.POINTER(KV), C.POINTER(Request), vp, vp, i32,
                                        vp, vp, C.POINTER(vp), vp, i32, vp, vp, i32, C.c_float, vp, vp, vp, vp]
    lib.acache_denoise_step.restype = C.c_int
    lib.acache_denoise_step_shared.argtypes = [vp, i32, C.POINTER(LayerWeights), C.POINTER(KV), C.POINTER(Request), vp, vp, i32,
                                               C.POINTER(vp), C.POINTER(vp), vp, vp, C.POINTER(vp), vp, i32, vp, vp, i32,
                                               C.c_float, vp, vp, vp, vp]
    lib.acache_denoise_step_shared.restype = C.c_int
    lib.acache_probe_select.argtypes = [vp, i32, C.POINTER(LayerWeights), C.POINTER(KV), C.POINTER(Request), vp,
                                        C.c_double, u32, vp, vp, vp, vp, vp]
    lib.acache_probe_select.restype = C.c_int
    lib.acache_commit_update.argtypes = [vp, vp, i32, vp, i32, i32, vp, vp, i32, C.c_float, vp, vp]
    lib.acache_commit_update.restype = C.c_int
    lib.acache_generate_block.argtypes = [vp, i32, C.POINTER(LayerWeights), C.POINTER(KV), C.POINTER(Request),
                                          C.POINTER(Request), vp, vp, i32, vp, vp, vp, vp, i32, vp, vp, i32, C.c_float,
                                          i32, i32, vp, vp, vp, vp, C.POINTER(i32), vp]
    lib.acache_generate_block.restype = C.c_int
    lib.acache_layer_step_shared.argtypes = [vp, C.POINTER(LayerWeights), C.POINTER(Request), C.POINTER(KV), vp, C.c_int,
                                             C.c_double, u32, vp, vp, vp, vp, vp, vp]
    lib.acache_layer_step_shared.restype = C.c_int
    lib.acache_recompute_rows_shared.argtypes = [vp, C.POINTER(LayerWeights), C.POINTER(Request), C.POINTER(Request),
                                                 C.POINTER(KV), vp, C.c_int, vp, i32, vp, vp, vp, vp, vp]
    lib.acache_recompute_rows_shared.restype = C.c_int
    lib.acache_decode_step_shared.argtypes = [vp, i32, C.POINTER(LayerWeights), C.POINTER(KV), C.POINTER(Request),
                                              C.POINTER(Request), vp, vp, i32, vp, C.POINTER(vp), C.POINTER(vp), vp, vp,
                                              C.POINTER(vp), vp, i32, vp, vp, i32, C.c_float, vp, vp, vp, vp]
    lib.acache_decode_step_shared.restype = C.c_int
    lib.acache_generate_block_shared.argtypes = [vp, i32, C.POINTER(LayerWeights), C.POINTER(KV), C.POINTER(Request),
                                                 C.POINTER(Request), vp, vp, i32, C.POINTER(vp), C.POINTER(vp), vp, vp, vp, vp,
                                                 i32, vp, vp, i32, C.c_float, i32, i32, vp, vp, vp, vp, C.POINTER(i32), vp]
    lib.acache_generate_block_shared.restype = C.c_int
    lib.acache_stage_timing.argtypes = [vp, C.c_int]
    lib.acache_stage_timing.restype = C.c_int
    lib.acache_read_stage_times.argtypes = [vp, C.POINTER(C.c_float)]
    lib.acache_read_stage_times.restype = C.c_int
    if path is None:
        _lib = lib
    return lib


def k_from_ratio(affix_len: int, ratio: float) -> int:
    return int(load_library().acache_k_from_ratio(int(affix_len), float(ratio)))


def score_anchors_static(desc: ModelDesc, req: Request, q_mask, kv: KV, scores, accumulate=False,
                         norm_full=False) -> int:
    """Scoring through the entry point that allocates nothing and needs no context or workspace
    (its scratch is a fixed array inside the library).  Returns the status code."""
    return int(load_library().acache_score_anchors_static(C.byref(desc), C.byref(req), _ptr(q_mask), C.byref(kv),
                                                          _ptr(scores), int(accumulate), int(norm_full), _stream()))


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a tensor, an int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream() -> int:
    import torch
    return torch.cuda.current_stream().cuda_stream


class Context:
    """One layer shape + workspace.  Mirrors the C entry points one to one."""

    def __init__(self, hidden, n_heads, n_kv_heads, head_dim, ffn, rms_eps, qkv_bias,
                 max_batch, max_ctx, max_affix, max_rows, max_masked, device="cuda:0", max_vocab=0, max_block=0):
        import torch
        self.lib = load_library()
        self.desc = ModelDesc(hidden, n_heads, n_kv_heads, head_dim, ffn, rms_eps, int(bool(qkv_bias)),
                              max_batch, max_ctx, max_affix, max_rows, max_masked, max_vocab, max_block)
        h = C.c_void_p()
        st = self.lib.acache_create(C.byref(self.desc), C.byref(h))
        if st != OK:
            raise AcacheError(st, "acache_create rejected the descriptor")
        self.h = h
        self.device = torch.device(device)
        nbytes = self.lib.acache_workspace_bytes(self.h)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) & ~255
            self._check(self.lib.acache_set_workspace(self.h, self._ws_ptr, nbytes, _stream()))
        self.workspace_bytes = nbytes

    @classmethod
    def for_shape(cls, shape, max_batch, max_ctx, max_affix, max_rows, max_masked, device="cuda:0", max_vocab=0,
                  max_block=0):
        return cls(shape.hidden, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.ffn, shape.rms_eps,
                   shape.qkv_bias, max_batch, max_ctx, max_affix, max_rows, max_masked, device, max_vocab, max_block)

    def close(self):
        if getattr(self, "h", None):
            self.lib.acache_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int):
        if st != OK:
            raise AcacheError(st, self.lib.acache_last_error(self.h).decode())

    # ---- marshalling helpers ----
    @staticmethod
    def weights(w: Dict[str, object]) -> LayerWeights:
        lw = LayerWeights()
        for name, _ in LayerWeights._fields_:
            setattr(lw, name, _ptr(w.get(name)))
        return lw

    @staticmethod
    def kv(cache_k, cache_v) -> KV:
        B, cap, hkv, d = cache_k.shape
        return KV(cache_k.data_ptr(), cache_v.data_ptr(), cap * hkv * d, cap)

    @staticmethod
    def request(batch, ctx_len, affix_start, affix_len, masked_pos, extra_rows, rope_cos, rope_sin,
                token_ids=None, n_embed=0) -> Request:
        nm = 0 if masked_pos is None else int(masked_pos.shape[1])
        ne = 0 if extra_rows is None else int(extra_rows.shape[1])
        return Request(batch, ctx_len, affix_start, affix_len, _ptr(masked_pos) if nm else None, nm,
                       _ptr(extra_rows) if ne else None, ne, _ptr(rope_cos), _ptr(rope_sin), _ptr(token_ids), n_embed)

    # ---- entry points ----
    def launch_count(self) -> int:
        return int(self.lib.acache_launch_count(self.h))

    def poll_status(self) -> int:
        flags = C.c_uint32(0)
        st = self.lib.acache_poll_status(self.h, _stream(), C.byref(flags))
        if st not in (OK, ERR_TIMEOUT):
            self._check(st)
        return int(flags.value)

    def poll_status_code(self):
        """(status code, flags) of acache_poll_status: ERR_TIMEOUT when a bounded device-side wait ran out."""
        flags = C.c_uint32(0)
        st = self.lib.acache_poll_status(self.h, _stream(), C.byref(flags))
        return int(st), int(flags.value)

    def debug_expire_next_wait(self):
        """Failure-detection self-test: the next Q/K/V projection's grid barrier is made to run out."""
        self._check(self.lib.acache_debug_expire_next_wait(self.h))

    def stage_timing(self, enable: bool):
        self._check(self.lib.acache_stage_timing(self.h, int(enable)))

    def read_stage_times(self) -> Dict[str, float]:
        """Milliseconds per stage of the last timed layer-step (synchronises)."""
        ms = (C.c_float * len(STAGES))()
        self._check(self.lib.acache_read_stage_times(self.h, ms))
        return {n: float(ms[i]) for i, n in enumerate(STAGES)}

    def score_anchors(self, req: Request, q_mask, kv: KV, scores, accumulate=False, norm_full=False):
        self._check(self.lib.acache_score_anchors(self.h, C.byref(req), _ptr(q_mask), C.byref(kv), _ptr(scores),
                                                  int(accumulate), int(norm_full), _stream()))

    def score_kv_deviation(self, req: Request, kv_ref: KV, kv_full: KV, scores, accumulate=False):
        self._check(self.lib.acache_score_kv_deviation(self.h, C.byref(req), C.byref(kv_ref), C.byref(kv_full), _ptr(scores),
                                                       int(accumulate), _stream()))

    def select_topk(self, scores, batch, affix_len, k, anchor_idx):
        self._check(self.lib.acache_select_topk(self.h, _ptr(scores), batch, affix_len, k, _ptr(anchor_idx), _stream()))

    def recompute_anchors(self, w: LayerWeights, req: Request, kv: KV, x, x_is_compact, anchor_idx, k,
                          k_new, v_new, y):
        self._check(self.lib.acache_recompute_anchors(self.h, C.byref(w), C.byref(req), C.byref(kv), _ptr(x),
                                                      int(x_is_compact), _ptr(anchor_idx), k, _ptr(k_new),
                                                      _ptr(v_new), _ptr(y), _stream()))

    def scatter_kv(self, req: Request, kv: KV, anchor_idx, k, k_new, v_new):
        self._check(self.lib.acache_scatter_kv(self.h, C.byref(req), C.byref(kv), _ptr(anchor_idx), k,
                                               _ptr(k_new), _ptr(v_new), _stream()))

    def layer_step(self, w: LayerWeights, req: Request, kv: KV, x, x_is_compact, ratio, flags, scores,
                   anchor_idx, y):
        self._check(self.lib.acache_layer_step(self.h, C.byref(w), C.byref(req), C.byref(kv), _ptr(x),
                                               int(x_is_compact), float(ratio), int(flags), _ptr(scores),
                                               _ptr(anchor_idx), _ptr(y), _stream()))

    def predict_commit(self, h, h_rows, block_rows, batch, n_blk, final_norm_g, w_lm, vocab, threshold, token,
                       confidence, commit):
        self._check(self.lib.acache_predict_commit(self.h, _ptr(h), h_rows, _ptr(block_rows), batch, n_blk,
                                                   _ptr(final_norm_g), _ptr(w_lm), vocab, float(threshold), _ptr(token),
                                                   _ptr(confidence), _ptr(commit), _stream()))

    def denoise_step(self, layers, kvs, req: Request, x0, anchor_idx, k, y_a, y_b, block_rows, n_blk, final_norm_g,
                     w_lm, vocab, threshold, token, confidence, commit) -> int:
        """layers: list of LayerWeights, kvs: list of KV.  Returns the device address of the last layer's output."""
        n = len(layers)
        la = (LayerWeights * n)(*layers)
        ka = (KV * n)(*kvs)
        last = C.c_void_p()
        self._check(self.lib.acache_denoise_step(self.h, n, la, ka, C.byref(req), _ptr(x0), _ptr(anchor_idx), k,
                                                 _ptr(y_a), _ptr(y_b), C.byref(last), _ptr(block_rows), n_blk,
                                                 _ptr(final_norm_g), _ptr(w_lm), vocab, float(threshold), _ptr(token),
                                                 _ptr(confidence), _ptr(commit), _stream()))
        return last.value

    def denoise_step_shared(self, layers, kvs, req: Request, x0, anchor_idx, k, k_new, v_new, y_a, y_b, block_rows, n_blk,
                            final_norm_g, w_lm, vocab, threshold, token, confidence, commit) -> int:
        """k_new, v_new: lists of per-layer tensors [B, K+e, Hkv, d].  Returns the device address of the last output."""
        n = len(layers)
        la = (LayerWeights * n)(*layers)
        ka = (KV * n)(*kvs)
        kn = (C.c_void_p * n)(*[_ptr(t) for t in k_new])
        vn = (C.c_void_p * n)(*[_ptr(t) for t in v_new])
        last = C.c_void_p()
        self._check(self.lib.acache_denoise_step_shared(self.h, n, la, ka, C.byref(req), _ptr(x0), _ptr(anchor_idx), k, kn, vn,
                                                        _ptr(y_a), _ptr(y_b), C.byref(last), _ptr(block_rows), n_blk,
                                                        _ptr(final_norm_g), _ptr(w_lm), vocab, float(threshold), _ptr(token),
                                                        _ptr(confidence), _ptr(commit), _stream()))
        return last.value

    def layer_step_shared(self, w: LayerWeights, req: Request, kv: KV, x, x_is_compact, ratio, flags, scores, anchor_idx,
                          k_new, v_new, y):
        """The fused layer-step over storage that is not written (the cache may be shared by the batch)."""
        self._check(self.lib.acache_layer_step_shared(self.h, C.byref(w), C.byref(req), C.byref(kv), _ptr(x), int(x_is_compact),
                                                      float(ratio), int(flags), _ptr(scores), _ptr(anchor_idx), _ptr(k_new),
                                                      _ptr(v_new), _ptr(y), _stream()))

    def recompute_rows_shared(self, w: LayerWeights, req_rows: Request, req_slots: Request, kv: KV, x, x_is_compact,
                              anchor_idx, k, slot_rows, k_slots, v_slots, y):
        self._check(self.lib.acache_recompute_rows_shared(self.h, C.byref(w), C.byref(req_rows), C.byref(req_slots),
                                                          C.byref(kv), _ptr(x), int(x_is_compact), _ptr(anchor_idx), k,
                                                          _ptr(slot_rows), _ptr(k_slots), _ptr(v_slots), _ptr(y), _stream()))

    def decode_step_shared(self, layers, kvs, req_rows: Request, req_slots: Request, x0, anchor_idx, k, slot_rows, k_slots,
                           v_slots, y_a, y_b, block_rows, n_blk, final_norm_g, w_lm, vocab, threshold, token, confidence,
                           commit) -> int:
        """k_slots, v_slots: lists of per-layer tensors [B, K+e, Hkv, d] as the refresh pass left them."""
        n = len(layers)
        la = (LayerWeights * n)(*layers)
        ka = (KV * n)(*kvs)
        kn = (C.c_void_p * n)(*[_ptr(t) for t in k_slots])
        vn = (C.c_void_p * n)(*[_ptr(t) for t in v_slots])
        last = C.c_void_p()
        self._check(self.lib.acache_decode_step_shared(self.h, n, la, ka, C.byref(req_rows), C.byref(req_slots), _ptr(x0),
                                                       _ptr(anchor_idx), k, _ptr(slot_rows), kn, vn, _ptr(y_a), _ptr(y_b),
                                                       C.byref(last), _ptr(block_rows), n_blk, _ptr(final_norm_g), _ptr(w_lm),
                                                       vocab, float(threshold), _ptr(token), _ptr(confidence), _ptr(commit),
                                                       _stream()))
        return last.value

    def generate_block_shared(self, layers, kvs, req_refresh: Request, req_decode: Request, embed, anchor_idx, k, k_slots,
                              v_slots, y_a, y_b, block_rows_refresh, block_rows_decode, n_blk, final_norm_g, w_lm, vocab,
                              threshold, mask_id, max_steps, token, confidence, commit, remaining) -> int:
        """acache_generate_block over shared affix storage; returns the number of model passes run."""
        n = len(layers)
        la = (LayerWeights * n)(*layers)
        ka = (KV * n)(*kvs)
        kn = (C.c_void_p * n)(*[_ptr(t) for t in k_slots])
        vn = (C.c_void_p * n)(*[_ptr(t) for t in v_slots])
        steps = C.c_int32(0)
        self._check(self.lib.acache_generate_block_shared(self.h, n, la, ka, C.byref(req_refresh), C.byref(req_decode),
                                                          _ptr(embed), _ptr(anchor_idx), k, kn, vn, _ptr(y_a), _ptr(y_b),
                                                          _ptr(block_rows_refresh), _ptr(block_rows_decode), n_blk,
                                                          _ptr(final_norm_g), _ptr(w_lm), vocab, float(threshold),
                                                          int(mask_id), int(max_steps), _ptr(token), _ptr(confidence),
                                                          _ptr(commit), _ptr(remaining), C.byref(steps), _stream()))
        return int(steps.value)

    def probe_select(self, layers, kvs, req: Request, x0, ratio, flags, y_a, y_b, scores, anchor_idx):
        n = len(layers)
        la = (LayerWeights * n)(*layers)
        ka = (KV * n)(*kvs)
        self._check(self.lib.acache_probe_select(self.h, n, la, ka, C.byref(req), _ptr(x0), float(ratio), int(flags),
                                                 _ptr(y_a), _ptr(y_b), _ptr(scores), _ptr(anchor_idx), _stream()))

    def commit_update(self, token_ids, ctx_len, block_pos, batch, n_blk, token, confidence, mask_id, threshold, remaining):
        self._check(self.lib.acache_commit_update(self.h, _ptr(token_ids), ctx_len, _ptr(block_pos), batch, n_blk,
                                                  _ptr(token), _ptr(confidence), int(mask_id), float(threshold),
                                                  _ptr(remaining), _stream()))

    def generate_block(self, layers, kvs, req_refresh: Request, req_decode: Request, embed, anchor_idx, k, y_a, y_b,
                       block_rows_refresh, block_rows_decode, n_blk, final_norm_g, w_lm, vocab, threshold, mask_id,
                       max_steps, token, confidence, commit, remaining) -> int:
        """Returns the number of model passes run (synchronises the stream once per pass)."""
        n = len(layers)
        la = (LayerWeights * n)(*layers)
        ka = (KV * n)(*kvs)
        steps = C.c_int32(0)
        self._check(self.lib.acache_generate_block(self.h, n, la, ka, C.byref(req_refresh), C.byref(req_decode), _ptr(embed),
                                                   _ptr(anchor_idx), k, _ptr(y_a), _ptr(y_b), _ptr(block_rows_refresh),
                                                   _ptr(block_rows_decode), n_blk, _ptr(final_norm_g), _ptr(w_lm), vocab,
                                                   float(threshold), int(mask_id), int(max_steps), _ptr(token),
                                                   _ptr(confidence), _ptr(commit), _ptr(remaining), C.byref(steps),
                                                   _stream()))
        return int(steps.value)

    def layer_step_host(self, w: LayerWeights, req: Request, kv: KV, x_host, ratio, flags, scores_host,
                        anchor_idx_host, y_host):
        self._check(self.lib.acache_layer_step_host(self.h, C.byref(w), C.byref(req), C.byref(kv), _ptr(x_host),
                                                    float(ratio), int(flags), _ptr(scores_host),
                                                    _ptr(anchor_idx_host), _ptr(y_host), _stream()))


    def host_x_in_place(self, x_host) -> bool:
        """True when layer_step_host reads this x in place (page-locked memory) instead of staging a copy."""
        return bool(self.lib.acache_host_x_in_place(_ptr(x_host)))


# --------------------------------------------------------------------------
# host <-> device conveniences for bf16-bit numpy arrays
# --------------------------------------------------------------------------
def to_device_bf16(bits, device="cuda:0"):
    """numpy uint16 bf16 bits -> torch.bfloat16 CUDA tensor (same bytes)."""
    import numpy as np
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def to_host_bits(t):
    """torch.bfloat16 tensor -> numpy uint16 bf16 bits."""
    import numpy as np
    import torch
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
