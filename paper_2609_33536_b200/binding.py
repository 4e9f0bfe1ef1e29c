"""ctypes binding of libekv.so: same entry-point names as include/ekv.h, argument marshalling
only. Device buffers are torch CUDA tensors (torch is used for memory and streams, nothing
else); every step of the path runs in the library's kernels. There is no fallback: a missing
library or a non-zero status raises."""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libekv.so")

EKV_TARGET, EKV_BASE = 0, 1
EXPORTS = ("ekv_version", "ekv_status_string", "ekv_set_option", "ekv_set_profile_events", "ekv_attn_workspace_bytes",
           "ekv_attn_decode", "ekv_attn_prefill_chunk", "ekv_downgrade", "ekv_refine",
           "ekv_validate_batch", "ekv_attn_decode_noalloc", "ekv_attn_decode_noalloc_max_bytes",
           "ekv_prefill_status", "ekv_lower_metadata", "ekv_attn_decode_structured",
           "ekv_kv_append", "ekv_lower_sparse_metadata", "ekv_reset_tags", "ekv_decode_status")


class EkvError(RuntimeError):
    pass


class ekv_pool(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("tags", C.c_void_p),
                ("num_blocks", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_size", C.c_int32), ("num_layers", C.c_int32), ("elem_type", C.c_int32),
                ("layer_stride_bytes", C.c_int64)]


EKV_BF16 = 0     # ekv_pool.elem_type: what the pool's 16-bit words (and q / out) are
EKV_FP16 = 1


class ekv_batch(C.Structure):
    _fields_ = [("block_table", C.c_void_p), ("seq_lens", C.c_void_p), ("batch", C.c_int32),
                ("max_blocks", C.c_int32), ("has_base", C.c_int32), ("reserved_", C.c_int32)]


_lib = None


def load(path: str | None = None):
    """Load the C-ABI library (no GPU needed to load it or to look up symbols)."""
    global _lib
    if _lib is None or path is not None:
        p = path or LIB_PATH
        if not os.path.exists(p):
            raise EkvError(f"{p} is missing: build it with `python -m paper_2609_33536_b200.build` "
                           "(there is no CPU fallback)")
        L = C.CDLL(p)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
        PP, BP = C.POINTER(ekv_pool), C.POINTER(ekv_batch)
        L.ekv_version.restype = C.c_int
        L.ekv_status_string.restype = C.c_char_p
        L.ekv_status_string.argtypes = [C.c_int]
        L.ekv_set_option.restype = C.c_int
        L.ekv_set_option.argtypes = [C.c_char_p, i64]
        L.ekv_set_profile_events.restype = C.c_int
        L.ekv_set_profile_events.argtypes = [vp, vp]
        L.ekv_attn_workspace_bytes.restype = sz
        L.ekv_attn_workspace_bytes.argtypes = [PP, i32, i32, i32, i32]
        L.ekv_attn_decode.restype = C.c_int
        L.ekv_attn_decode.argtypes = [PP, i32, BP, vp, vp, i32, f32, i32, vp, sz, vp]
        L.ekv_attn_decode_noalloc.restype = C.c_int
        L.ekv_attn_decode_noalloc.argtypes = [PP, i32, BP, vp, vp, i32, f32, i32, vp]
        L.ekv_attn_decode_noalloc_max_bytes.restype = sz
        L.ekv_attn_prefill_chunk.restype = C.c_int
        L.ekv_attn_prefill_chunk.argtypes = [PP, i32, BP, vp, vp, vp, i32, f32, i32, i32, i32, vp, sz, vp]
        L.ekv_downgrade.restype = C.c_int
        L.ekv_downgrade.argtypes = [PP, BP, i32, vp, vp, vp, vp, vp, vp, vp]
        L.ekv_refine.restype = C.c_int
        L.ekv_refine.argtypes = [PP, BP, i32, vp, vp, vp, vp, vp, vp, vp]
        L.ekv_lower_metadata.restype = C.c_int
        L.ekv_lower_metadata.argtypes = [PP, BP, vp, vp, vp]
        L.ekv_attn_decode_structured.restype = C.c_int
        L.ekv_attn_decode_structured.argtypes = [PP, i32, BP, vp, vp, vp, i32, f32, i32, vp, sz, vp]
        L.ekv_kv_append.restype = C.c_int
        L.ekv_kv_append.argtypes = [PP, i32, BP, vp, vp, vp, i32, vp, vp]
        L.ekv_lower_sparse_metadata.restype = C.c_int
        L.ekv_lower_sparse_metadata.argtypes = [PP, BP, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        L.ekv_reset_tags.restype = C.c_int
        L.ekv_reset_tags.argtypes = [PP, vp, i32, vp]
        L.ekv_prefill_status.restype = C.c_int
        L.ekv_decode_status.restype = C.c_int
        L.ekv_validate_batch.restype = C.c_int
        L.ekv_validate_batch.argtypes = [PP, BP, vp, vp]
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        raise EkvError(f"{what}: {load().ekv_status_string(rc).decode()} ({rc})")


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise EkvError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


class Pool:
    """Device KV pool: K and V tensors [layers][num_blocks][Hkv*16*D] (int16 words or bf16),
    uint8 tags [num_blocks]. Holds references to the tensors and the C struct."""

    def __init__(self, k_pool, v_pool, tags, num_kv_heads: int, head_dim: int, page_size: int = 16,
                 elem_type: int = EKV_BF16):
        assert k_pool.dim() == 3 and k_pool.shape == v_pool.shape and k_pool.element_size() == 2
        self.k_pool, self.v_pool, self.tags = k_pool, v_pool, tags
        self.num_layers, self.num_blocks, words = k_pool.shape
        assert words == num_kv_heads * page_size * head_dim
        self.num_kv_heads, self.head_dim, self.page_size = num_kv_heads, head_dim, page_size
        self.block_bytes = words * 2
        self.elem_type = int(elem_type)
        self.c = ekv_pool(_ptr(k_pool), _ptr(v_pool), _ptr(tags), self.num_blocks, num_kv_heads, head_dim,
                          page_size, self.num_layers, self.elem_type, self.num_blocks * self.block_bytes)

    def new_resid(self, n_slots: int):
        """Residual (low byte) buffer for one tensor: [slots][layers][block_bytes] bytes."""
        return torch.zeros((n_slots, self.num_layers, self.block_bytes), dtype=torch.uint8, device=self.k_pool.device)


class Batch:
    """Device batch metadata: int32 block_table [batch][max_blocks], int32 seq_lens [batch]."""

    def __init__(self, block_table, seq_lens, has_base: bool):
        assert block_table.dtype == torch.int32 and seq_lens.dtype == torch.int32
        self.block_table, self.seq_lens = block_table, seq_lens
        self.batch, self.max_blocks = block_table.shape
        self.c = ekv_batch(_ptr(block_table), _ptr(seq_lens), self.batch, self.max_blocks, int(has_base), 0)

    @property
    def has_base(self) -> bool:
        return bool(self.c.has_base)

    @has_base.setter
    def has_base(self, v: bool):
        self.c.has_base = int(v)


def ekv_version() -> int:
    return int(load().ekv_version())


def ekv_set_option(name: str, value: int):
    _check(load().ekv_set_option(name.encode(), int(value)), "ekv_set_option")


def ekv_set_profile_events(ev_begin=None, ev_end=None):
    """torch.cuda.Event(enable_timing=True) pair recorded around the main kernel of later calls
    (None, None switches the hook off). The events must have been created (recorded once)."""
    hb = ev_begin.cuda_event if ev_begin is not None else None
    he = ev_end.cuda_event if ev_end is not None else None
    _check(load().ekv_set_profile_events(hb, he), "ekv_set_profile_events")


def ekv_attn_workspace_bytes(pool: Pool, batch: int, num_q_heads: int, max_seq_len: int, total_q: int = 0) -> int:
    return int(load().ekv_attn_workspace_bytes(C.byref(pool.c), batch, num_q_heads, max_seq_len, total_q))


def new_workspace(pool: Pool, batch: int, num_q_heads: int, max_seq_len: int, total_q: int = 0):
    n = ekv_attn_workspace_bytes(pool, batch, num_q_heads, max_seq_len, total_q)
    return torch.empty(max(n, 256), dtype=torch.uint8, device=pool.k_pool.device)


def ekv_attn_decode(pool: Pool, layer: int, batch: Batch, q, out, num_q_heads: int, sm_scale: float,
                    max_seq_len: int, workspace):
    _check(load().ekv_attn_decode(C.byref(pool.c), layer, C.byref(batch.c), _ptr(q), _ptr(out), num_q_heads,
                                  float(sm_scale), int(max_seq_len), _ptr(workspace),
                                  workspace.numel() if workspace is not None else 0, _stream()),
           "ekv_attn_decode")


def ekv_lower_metadata(pool: Pool, batch: Batch, boundaries, flags):
    """boundaries: int32 [batch][2] out; flags: int32 [2] out (has_base, any_irregular)."""
    _check(load().ekv_lower_metadata(C.byref(pool.c), C.byref(batch.c), _ptr(boundaries), _ptr(flags), _stream()),
           "ekv_lower_metadata")


def ekv_lower_sparse_metadata(pool: Pool, batch: Batch, seq_lens_out, row_of, lens, blk_start, blk_ids,
                              range_start, ranges, boundaries, flags):
    """Scheduler-side sparse description (block lists + BASE pair ranges, CSR) -> block-table rows,
    sequence lengths, boundaries [batch][2], flags [4] (any BASE, any irregular, disagreeing pairs,
    n_req - first disagreeing request)."""
    _check(load().ekv_lower_sparse_metadata(C.byref(pool.c), C.byref(batch.c), _ptr(seq_lens_out), int(lens.numel()),
                                            _ptr(row_of), _ptr(lens), _ptr(blk_start), _ptr(blk_ids), _ptr(range_start),
                                            _ptr(ranges), _ptr(boundaries), _ptr(flags), _stream()),
           "ekv_lower_sparse_metadata")


def ekv_reset_tags(pool: Pool, block_ids):
    """tags[block_ids] = TARGET for blocks that leave their request."""
    _check(load().ekv_reset_tags(C.byref(pool.c), _ptr(block_ids), int(block_ids.numel()), _stream()), "ekv_reset_tags")


def ekv_attn_decode_structured(pool: Pool, layer: int, batch: Batch, boundaries, q, out, num_q_heads: int,
                               sm_scale: float, max_seq_len: int, workspace):
    _check(load().ekv_attn_decode_structured(C.byref(pool.c), layer, C.byref(batch.c), _ptr(boundaries), _ptr(q),
                                             _ptr(out), num_q_heads, float(sm_scale), int(max_seq_len), _ptr(workspace),
                                             workspace.numel() if workspace is not None else 0, _stream()),
           "ekv_attn_decode_structured")


def ekv_attn_decode_noalloc(pool: Pool, layer: int, batch: Batch, q, out, num_q_heads: int, sm_scale: float,
                            max_seq_len: int):
    """Decode attention for callers that cannot allocate device memory: no workspace argument,
    the split-K partials use a fixed 16 MiB array inside the library. Shapes that need more are
    refused (EkvError, 'workspace ...'). Calls that overlap on the GPU race on that array."""
    _check(load().ekv_attn_decode_noalloc(C.byref(pool.c), layer, C.byref(batch.c), _ptr(q), _ptr(out), num_q_heads,
                                          float(sm_scale), int(max_seq_len), _stream()),
           "ekv_attn_decode_noalloc")


def ekv_attn_decode_noalloc_max_bytes() -> int:
    return int(load().ekv_attn_decode_noalloc_max_bytes())


def ekv_attn_prefill_chunk(pool: Pool, layer: int, batch: Batch, q_start, q, out, num_q_heads: int,
                           sm_scale: float, total_q: int, max_q_len: int, max_seq_len: int, workspace):
    _check(load().ekv_attn_prefill_chunk(C.byref(pool.c), layer, C.byref(batch.c), _ptr(q_start), _ptr(q), _ptr(out),
                                         num_q_heads, float(sm_scale), int(total_q), int(max_q_len),
                                         int(max_seq_len), _ptr(workspace),
                                         workspace.numel() if workspace is not None else 0, _stream()),
           "ekv_attn_prefill_chunk")


def ekv_kv_append(pool: Pool, layer: int, batch: Batch, q_start, k_new, v_new, dev_status=None):
    """Write the new tokens' K/V (bf16 [total][Hkv][D]) into their TARGET blocks."""
    _check(load().ekv_kv_append(C.byref(pool.c), layer, C.byref(batch.c), _ptr(q_start), _ptr(k_new), _ptr(v_new),
                                int(k_new.shape[0]), _ptr(dev_status), _stream()),
           "ekv_kv_append")


def ekv_decode_status() -> int:
    """Status word of the TMA-staged decode kernel (synchronises; 0 = ok); clears it."""
    return int(load().ekv_decode_status())


def ekv_prefill_status() -> int:
    """Status word of the tensor-core prefill kernel (synchronises; 0 = ok); clears it."""
    return int(load().ekv_prefill_status())


def ekv_downgrade(pool: Pool, batch: Batch, pair_req, pair_idx, k_resid, v_resid, resid_slot, freed_blocks_out):
    n = int(pair_req.numel())
    _check(load().ekv_downgrade(C.byref(pool.c), C.byref(batch.c), n, _ptr(pair_req), _ptr(pair_idx),
                                _ptr(k_resid), _ptr(v_resid), _ptr(resid_slot), _ptr(freed_blocks_out), _stream()),
           "ekv_downgrade")


def ekv_refine(pool: Pool, batch: Batch, pair_req, pair_idx, new_blocks, k_resid, v_resid, resid_slot):
    n = int(pair_req.numel())
    _check(load().ekv_refine(C.byref(pool.c), C.byref(batch.c), n, _ptr(pair_req), _ptr(pair_idx), _ptr(new_blocks),
                             _ptr(k_resid), _ptr(v_resid), _ptr(resid_slot), _stream()),
           "ekv_refine")


def ekv_validate_batch(pool: Pool, batch: Batch, dev_status):
    _check(load().ekv_validate_batch(C.byref(pool.c), C.byref(batch.c), _ptr(dev_status), _stream()),
           "ekv_validate_batch")


# ---- glue used by tests / benchmark / smoke: upload a generated workload ----------------------

def upload(wl, device="cuda"):
    """Workload (host numpy arrays, all-TARGET) -> (Pool, Batch, q tensor) on the device."""
    import numpy as np
    dev = torch.device(device)
    k = torch.from_numpy(wl.k_pool.view(np.int16)).to(dev)
    v = torch.from_numpy(wl.v_pool.view(np.int16)).to(dev)
    tags = torch.zeros(wl.num_blocks, dtype=torch.uint8, device=dev)
    fp16 = getattr(wl, "elem_type", "bf16") == "fp16"
    pool = Pool(k, v, tags, wl.num_kv_heads, wl.head_dim, wl.page_size, elem_type=EKV_FP16 if fp16 else EKV_BF16)
    bt = torch.from_numpy(wl.block_table).to(dev)
    sl = torch.from_numpy(wl.seq_lens).to(dev)
    batch = Batch(bt, sl, has_base=False)
    q = torch.from_numpy(wl.q.view(np.int16)).to(dev).view(torch.float16 if fp16 else torch.bfloat16)
    return pool, batch, q
