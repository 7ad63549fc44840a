"""Thin ctypes binding of libpsmc.so: same names as include/psmc.h, argument marshalling only.

Every step of the path runs in the CUDA kernels of the library; nothing here computes.  The
library must have been built (``python -m paper_2602_10273_b200.build``); a missing or unloadable
library is an error, never a reason to fall back to anything else.  torch supplies device memory
and the stream: tensors are passed as ``data_ptr()``, the stream as ``cuda_stream``.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

OK, E_INVAL, E_NOMEM, E_CUDA, E_STATE, E_NUMERIC, E_TIMEOUT, E_HAZARD, E_TOO_LARGE = range(9)
STATIC_SCRATCH_BYTES = 4 << 20
F32, BF16 = 0, 1
SYSTEMATIC, STRATIFIED, MULTINOMIAL, RESIDUAL = 0, 1, 2, 3

_lib = None


class PsmcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().psmc_strerror(code).decode() if _lib is not None else str(code)
        super().__init__("%s: %s (status %d)" % (where, msg, code))


class KvDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("k", C.POINTER(C.c_void_p)), ("v", C.POINTER(C.c_void_p)),
                ("n_kv_heads", C.c_int), ("head_dim", C.c_int), ("max_len", C.c_int), ("dt", C.c_int),
                ("stride_row", C.c_int64), ("stride_head", C.c_int64), ("skip_shared_prompt", C.c_int)]


class KvPools(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("k", C.POINTER(C.c_void_p)), ("v", C.POINTER(C.c_void_p)),
                ("n_kv_heads", C.c_int), ("head_dim", C.c_int), ("dt", C.c_int)]


def lib():
    """Load libpsmc.so (once).  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(_build.LIB):
            raise ImportError("libpsmc.so is missing at %s: run `python -m paper_2602_10273_b200.build` "
                              "(nvcc, sm_100a); this package has no CPU or eager fallback" % _build.LIB)
        L = C.CDLL(_build.LIB)
        vp, i32p, f64p, u8p = C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p
        L.psmc_init.restype = C.c_int
        L.psmc_init.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_float, C.c_float, C.c_float, C.c_int,
                                C.c_uint64, C.c_int]
        L.psmc_init_batched.restype = C.c_int
        L.psmc_init_batched.argtypes = [C.POINTER(vp), C.c_int, C.c_int, C.c_int, C.c_float, C.c_float, C.c_float,
                                        C.c_int, C.c_uint64, C.c_int, C.c_int, C.POINTER(C.c_int32)]
        L.psmc_destroy.restype = C.c_int
        L.psmc_destroy.argtypes = [vp]
        L.psmc_set_resampler.restype = C.c_int
        L.psmc_set_resampler.argtypes = [vp, C.c_int]
        L.psmc_set_proposal_mask.restype = C.c_int
        L.psmc_set_proposal_mask.argtypes = [vp, C.c_int, C.c_double]
        L.psmc_reset.restype = C.c_int
        L.psmc_reset.argtypes = [vp, C.c_uint64]
        L.psmc_step.restype = C.c_int
        L.psmc_step.argtypes = [vp, vp, C.c_int, C.c_int64, vp]
        L.psmc_step_host.restype = C.c_int
        L.psmc_step_host.argtypes = [vp, vp, C.c_int, C.c_int64, vp, vp]
        L.psmc_logits_pass_scratch_bytes.restype = C.c_size_t
        L.psmc_logits_pass_scratch_bytes.argtypes = [C.c_int, C.c_int]
        L.psmc_step_layout.restype = C.c_int
        L.psmc_step_layout.argtypes = [C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_int]
        L.psmc_step_share_of.restype = C.c_int
        L.psmc_step_share_of.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int]
        L.psmc_logits_pass.restype = C.c_int
        L.psmc_logits_pass.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_double, C.c_double, f64p, u8p,
                                       vp, C.c_size_t, i32p, f64p, f64p, i32p, vp]
        L.psmc_logits_pass_static.restype = C.c_int
        L.psmc_logits_pass_static.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_double, C.c_double, f64p,
                                              u8p, i32p, f64p, f64p, i32p, vp]
        L.psmc_reindex_kv.restype = C.c_int
        L.psmc_reindex_kv.argtypes = [vp, C.POINTER(KvDesc), C.POINTER(KvDesc), i32p, vp]
        L.psmc_select.restype = C.c_int
        L.psmc_select.argtypes = [vp, i32p, i32p, i32p, vp]
        for name in ("psmc_tokens", "psmc_last_tokens", "psmc_log_weights", "psmc_log_inc", "psmc_logp_tok",
                     "psmc_cum_logp", "psmc_ancestors", "psmc_slot_map", "psmc_resampled", "psmc_ess",
                     "psmc_log_z", "psmc_lens", "psmc_done", "psmc_move_count", "psmc_mask_sizes"):
            f = getattr(L, name)
            f.restype = C.c_void_p
            f.argtypes = [vp]
        L.psmc_step_index.restype = C.c_int
        L.psmc_step_index.argtypes = [vp]
        L.psmc_rows.restype = C.c_int
        L.psmc_rows.argtypes = [vp]
        L.psmc_set_state.restype = C.c_int
        L.psmc_set_state.argtypes = [vp, vp, vp, vp, vp]
        L.psmc_sync_status.restype = C.c_int
        L.psmc_sync_status.argtypes = [vp, vp]
        L.psmc_kv_paged_create.restype = C.c_int
        L.psmc_kv_paged_create.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int]
        L.psmc_kv_paged_append.restype = C.c_int
        L.psmc_kv_paged_append.argtypes = [vp, vp]
        L.psmc_reindex_kv_paged.restype = C.c_int
        L.psmc_reindex_kv_paged.argtypes = [vp, C.POINTER(KvPools), vp]
        for name in ("psmc_kv_paged_table", "psmc_kv_paged_refcount", "psmc_kv_paged_free_count"):
            getattr(L, name).restype = C.c_void_p
            getattr(L, name).argtypes = [vp]
        L.psmc_shard_sweep.restype = C.c_int
        L.psmc_shard_sweep.argtypes = [vp, vp, C.c_int, C.c_int64, C.c_int, vp, vp]
        L.psmc_shard_locate.restype = C.c_int
        L.psmc_shard_locate.argtypes = [vp, C.c_int, vp, C.c_int, C.c_int, vp, vp]
        L.psmc_shard_finish.restype = C.c_int
        L.psmc_shard_finish.argtypes = [vp, vp, vp, C.c_int, vp]
        L.psmc_tiles_feed.restype = C.c_int
        L.psmc_tiles_feed.argtypes = [vp, vp, C.c_int, C.c_int64, C.c_int, C.c_int, vp]
        L.psmc_tiles_need.restype = C.c_int
        L.psmc_tiles_need.argtypes = [vp, vp, vp]
        L.psmc_tiles_finish.restype = C.c_int
        L.psmc_tiles_finish.argtypes = [vp, vp, C.c_int, C.c_int64, vp]
        L.psmc_state_bytes.restype = C.c_size_t
        L.psmc_state_bytes.argtypes = [vp]
        L.psmc_state_save.restype = C.c_int
        L.psmc_state_save.argtypes = [vp, vp, C.c_size_t]
        L.psmc_state_load.restype = C.c_int
        L.psmc_state_load.argtypes = [vp, vp, C.c_size_t]
        L.psmc_timing_enable.restype = C.c_int
        L.psmc_timing_enable.argtypes = [vp, C.c_int]
        L.psmc_timing_read.restype = C.c_int
        L.psmc_timing_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.psmc_strerror.restype = C.c_char_p
        L.psmc_strerror.argtypes = [C.c_int]
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != OK:
        raise PsmcError(code, where)


def _ptr(t) -> int:
    """Device or host address of a tensor / numpy array / raw int (None -> NULL)."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    raise TypeError(type(t))


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("logits / KV must be float32 or bfloat16, got %s" % t.dtype)


_VIEW_DTYPES = {"psmc_tokens": torch.int32, "psmc_last_tokens": torch.int32, "psmc_log_weights": torch.float64,
                "psmc_log_inc": torch.float64, "psmc_logp_tok": torch.float64, "psmc_cum_logp": torch.float64,
                "psmc_ancestors": torch.int32, "psmc_slot_map": torch.int32, "psmc_resampled": torch.int32,
                "psmc_ess": torch.float64, "psmc_log_z": torch.float64, "psmc_lens": torch.int32,
                "psmc_mask_sizes": torch.int32, "psmc_done": torch.uint8, "psmc_move_count": torch.int32, "psmc_kv_paged_table": torch.int32,
                "psmc_kv_paged_refcount": torch.int32, "psmc_kv_paged_free_count": torch.int32}


_TYPESTR = {torch.int32: "<i4", torch.float64: "<f8", torch.uint8: "|u1"}


class _DevArray:
    """Minimal __cuda_array_interface__ carrier so torch can wrap a raw device pointer."""

    def __init__(self, addr: int, n: int, dtype: torch.dtype):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": _TYPESTR[dtype], "data": (addr, False),
                                         "version": 2, "strides": None}


class Psmc:
    """Handle on a psmc_ctx.  Methods carry the C names without the prefix."""

    def __init__(self, N, V, alpha, tau, ess_thresh, ramp, seed, eos_id, G=1, T_max=4096, prompt_len=None):
        self._h = C.c_void_p()
        self.G, self.N, self.V, self.R, self.T_max = G, N, V, G * N, T_max
        pl = None
        if prompt_len is not None:
            pl = np.ascontiguousarray(prompt_len, dtype=np.int32)
            assert pl.size == G
        code = lib().psmc_init_batched(C.byref(self._h), G, N, V, alpha, tau, ess_thresh, ramp, seed, eos_id, T_max,
                                       None if pl is None else pl.ctypes.data_as(C.POINTER(C.c_int32)))
        _check(code, "psmc_init_batched")
        self._kv_keepalive = None

    def destroy(self):
        if self._h:
            lib().psmc_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def set_resampler(self, kind: int) -> None:
        """psmc_set_resampler: SYSTEMATIC (default), STRATIFIED, MULTINOMIAL or RESIDUAL."""
        _check(lib().psmc_set_resampler(self._h, kind), "psmc_set_resampler")

    def set_proposal_mask(self, top_k: int = 0, top_p: float = 0.0) -> None:
        """psmc_set_proposal_mask: proposal restricted to the top_k tokens or to the nucleus of share top_p (0, 0 = off)."""
        _check(lib().psmc_set_proposal_mask(self._h, top_k, top_p), "psmc_set_proposal_mask")

    def reset(self, seed):
        _check(lib().psmc_reset(self._h, seed), "psmc_reset")

    def step(self, logits: torch.Tensor, stream=None):
        """logits: CUDA tensor [R, V] (float32 / bfloat16), unit stride along V."""
        assert logits.is_cuda and logits.dim() == 2 and logits.stride(1) == 1 and logits.shape == (self.R, self.V)
        _check(lib().psmc_step(self._h, logits.data_ptr(), _dtype_code(logits), logits.stride(0), _stream(stream)),
               "psmc_step")

    def step_host(self, logits: torch.Tensor, tokens_out: torch.Tensor, stream=None):
        """logits: HOST tensor [R, V] (ideally pinned); tokens_out: HOST int32 [R]."""
        assert not logits.is_cuda and not tokens_out.is_cuda and tokens_out.dtype == torch.int32
        assert logits.dim() == 2 and logits.stride(1) == 1 and logits.shape == (self.R, self.V)
        _check(lib().psmc_step_host(self._h, logits.data_ptr(), _dtype_code(logits), logits.stride(0),
                                    tokens_out.data_ptr(), _stream(stream)), "psmc_step_host")

    # ---- the step with the vocabulary split over ranks: three calls around two all-gathers made by the caller ----
    def shard_sweep(self, logits_local: torch.Tensor, triples_out: torch.Tensor, stream=None):
        """logits_local: CUDA [R, V_local] columns of this rank (unit stride along V); triples_out: CUDA float64 [R, 3]."""
        assert logits_local.is_cuda and logits_local.dim() == 2 and logits_local.stride(1) == 1
        assert logits_local.shape[0] == self.R
        assert triples_out.is_cuda and triples_out.dtype == torch.float64 and triples_out.is_contiguous()
        assert triples_out.numel() == 3 * self.R
        _check(lib().psmc_shard_sweep(self._h, logits_local.data_ptr(), _dtype_code(logits_local),
                                      logits_local.stride(0), logits_local.shape[1], triples_out.data_ptr(),
                                      _stream(stream)), "psmc_shard_sweep")

    def shard_locate(self, v0: int, all_triples: torch.Tensor, rank: int, picks_out: torch.Tensor, stream=None):
        """all_triples: CUDA float64 [P, R, 3] in rank order; picks_out: CUDA int32 [R, 2] (token id, logit bits)."""
        assert all_triples.is_cuda and all_triples.dtype == torch.float64 and all_triples.is_contiguous()
        assert all_triples.dim() == 3 and all_triples.shape[1:] == (self.R, 3)
        assert picks_out.is_cuda and picks_out.dtype == torch.int32 and picks_out.is_contiguous()
        assert picks_out.numel() == 2 * self.R
        _check(lib().psmc_shard_locate(self._h, v0, all_triples.data_ptr(), all_triples.shape[0], rank,
                                       picks_out.data_ptr(), _stream(stream)), "psmc_shard_locate")

    def shard_finish(self, all_triples: torch.Tensor, all_picks: torch.Tensor, stream=None):
        """all_picks: CUDA int32 [P, R, 2] in rank order."""
        assert all_picks.is_cuda and all_picks.dtype == torch.int32 and all_picks.is_contiguous()
        assert all_picks.dim() == 3 and all_picks.shape == (all_triples.shape[0], self.R, 2)
        _check(lib().psmc_shard_finish(self._h, all_triples.data_ptr(), all_picks.data_ptr(), all_triples.shape[0],
                                       _stream(stream)), "psmc_shard_finish")

    # ---- the step fed one vocabulary tile at a time: feed every tile in order, ask which tile each row needs again,
    # hand those tiles back
    def tiles_feed(self, tile: torch.Tensor, v0: int, stream=None):
        """tile: CUDA [R, width] logits of columns v0 .. v0+width (unit stride along the columns)."""
        assert tile.is_cuda and tile.dim() == 2 and tile.stride(1) == 1 and tile.shape[0] == self.R
        _check(lib().psmc_tiles_feed(self._h, tile.data_ptr(), _dtype_code(tile), tile.stride(0), v0, tile.shape[1],
                                     _stream(stream)), "psmc_tiles_feed")

    def tiles_need(self, first_column_out: torch.Tensor, stream=None):
        """first_column_out: CUDA int32 [R]: first column of the tile each row needs again (-1: finished row)."""
        assert first_column_out.is_cuda and first_column_out.dtype == torch.int32 and first_column_out.numel() == self.R
        _check(lib().psmc_tiles_need(self._h, first_column_out.data_ptr(), _stream(stream)), "psmc_tiles_need")

    def tiles_finish(self, row_tiles: torch.Tensor, stream=None):
        """row_tiles: CUDA [R, tile width]: row r holds its own row's logits from first_column[r] on (-inf past V)."""
        assert row_tiles.is_cuda and row_tiles.dim() == 2 and row_tiles.stride(1) == 1 and row_tiles.shape[0] == self.R
        _check(lib().psmc_tiles_finish(self._h, row_tiles.data_ptr(), _dtype_code(row_tiles), row_tiles.stride(0),
                                       _stream(stream)), "psmc_tiles_finish")

    def make_kv_desc(self, k_layers, v_layers, skip_shared_prompt: bool = False):
        """k_layers / v_layers: lists of CUDA tensors [R, H, max_len, D] with (max_len, D) contiguous.
        skip_shared_prompt: the rows of a group hold the same prompt positions, which then stay where they are."""
        k0 = k_layers[0]
        R, H, L, D = k0.shape
        assert R == self.R and k0.stride(3) == 1 and k0.stride(2) == D
        n = len(k_layers)
        ka = (C.c_void_p * n)(*[t.data_ptr() for t in k_layers])
        va = (C.c_void_p * n)(*[t.data_ptr() for t in v_layers])
        for t in list(k_layers) + list(v_layers):
            assert t.shape == k0.shape and t.stride() == k0.stride() and t.dtype == k0.dtype and t.is_cuda
        d = KvDesc(n, C.cast(ka, C.POINTER(C.c_void_p)), C.cast(va, C.POINTER(C.c_void_p)), H, D, L,
                   _dtype_code(k0), k0.stride(0), k0.stride(1), 1 if skip_shared_prompt else 0)
        d._keep = (ka, va, list(k_layers), list(v_layers))
        return d

    def reindex_kv(self, src: KvDesc, dst: KvDesc = None, idx_override: torch.Tensor = None, stream=None):
        if idx_override is not None:
            assert idx_override.is_cuda and idx_override.dtype == torch.int32 and idx_override.numel() == self.R
        _check(lib().psmc_reindex_kv(self._h, C.byref(src), None if dst is None else C.byref(dst),
                                     _ptr(idx_override), _stream(stream)), "psmc_reindex_kv")

    def state_save(self) -> bytes:
        """psmc_state_save: snapshot of the run (particle state, last results, ancestry log) as bytes."""
        n = lib().psmc_state_bytes(self._h)
        buf = C.create_string_buffer(n)
        _check(lib().psmc_state_save(self._h, buf, n), "psmc_state_save")
        return buf.raw

    def state_load(self, blob: bytes) -> None:
        """psmc_state_load: continue the run a snapshot was taken from (same G, N, V, T_max)."""
        _check(lib().psmc_state_load(self._h, blob, len(blob)), "psmc_state_load")

    # ---- paged KV cache (block table, copy on write)
    def kv_paged_create(self, n_blocks: int, block_len: int, max_blocks_per_row: int, share_prompt: bool = True):
        _check(lib().psmc_kv_paged_create(self._h, n_blocks, block_len, max_blocks_per_row, 1 if share_prompt else 0),
               "psmc_kv_paged_create")
        self._paged = (n_blocks, block_len, max_blocks_per_row)

    def kv_paged_append(self, stream=None):
        _check(lib().psmc_kv_paged_append(self._h, _stream(stream)), "psmc_kv_paged_append")

    def make_kv_pools(self, k_pools, v_pools):
        """k_pools / v_pools: lists (one per layer) of contiguous CUDA tensors [n_blocks, H, block_len, D]."""
        p0 = k_pools[0]
        nb, H, Bl, D = p0.shape
        assert (nb, Bl) == self._paged[:2]
        n = len(k_pools)
        for t in list(k_pools) + list(v_pools):
            assert t.shape == p0.shape and t.is_contiguous() and t.dtype == p0.dtype and t.is_cuda
        ka = (C.c_void_p * n)(*[t.data_ptr() for t in k_pools])
        va = (C.c_void_p * n)(*[t.data_ptr() for t in v_pools])
        d = KvPools(n, C.cast(ka, C.POINTER(C.c_void_p)), C.cast(va, C.POINTER(C.c_void_p)), H, D, _dtype_code(p0))
        d._keep = (ka, va, list(k_pools), list(v_pools))
        return d

    def reindex_kv_paged(self, pools: KvPools, stream=None):
        _check(lib().psmc_reindex_kv_paged(self._h, C.byref(pools), _stream(stream)), "psmc_reindex_kv_paged")

    kv_paged_table = property(lambda s: s.device_view("psmc_kv_paged_table", s.R * s._paged[2]).view(s.R, s._paged[2]))
    kv_paged_refcount = property(lambda s: s.device_view("psmc_kv_paged_refcount", s._paged[0]))
    kv_paged_free_count = property(lambda s: int(s._view("psmc_kv_paged_free_count", 1)[0]))

    def select(self, out_tokens=None, out_len=None, out_index=None, stream=None):
        dev = torch.device("cuda", torch.cuda.current_device())
        if out_tokens is None:
            out_tokens = torch.empty((self.G, self.T_max), dtype=torch.int32, device=dev)
        if out_len is None:
            out_len = torch.empty(self.G, dtype=torch.int32, device=dev)
        if out_index is None:
            out_index = torch.empty(self.G, dtype=torch.int32, device=dev)
        _check(lib().psmc_select(self._h, out_tokens.data_ptr(), out_len.data_ptr(), out_index.data_ptr(),
                                 _stream(stream)), "psmc_select")
        return out_tokens, out_len, out_index

    def set_state(self, log_w=None, cum_logp=None, done=None, lens=None):
        a = None if log_w is None else np.ascontiguousarray(log_w, dtype=np.float64)
        b = None if cum_logp is None else np.ascontiguousarray(cum_logp, dtype=np.float64)
        c = None if done is None else np.ascontiguousarray(done, dtype=np.uint8)
        d = None if lens is None else np.ascontiguousarray(lens, dtype=np.int32)
        _check(lib().psmc_set_state(self._h, _ptr(a), _ptr(b), _ptr(c), _ptr(d)), "psmc_set_state")

    def timing_enable(self, on):
        """False/0: off; True/1: one event bracket per kernel; 2: one per psmc_step call and one per reindex kernel."""
        _check(lib().psmc_timing_enable(self._h, int(on)), "psmc_timing_enable")

    def timing_read(self):
        """(ms[3], launches[3]) for the logit pass, the weights/resampling kernel and the KV reindex."""
        ms, n = (C.c_double * 3)(), (C.c_int64 * 3)()
        _check(lib().psmc_timing_read(self._h, ms, n), "psmc_timing_read")
        return list(ms), list(n)

    def sync_status(self, stream=None) -> int:
        return lib().psmc_sync_status(self._h, _stream(stream))

    @property
    def step_index(self) -> int:
        return lib().psmc_step_index(self._h)

    def device_view(self, name: str, n: int) -> torch.Tensor:
        """The library-owned device array behind a view accessor, wrapped (not copied) as a CUDA tensor."""
        addr = getattr(lib(), name)(self._h)
        return torch.as_tensor(_DevArray(addr, n, _VIEW_DTYPES[name]), device="cuda")

    def _view(self, name: str, n: int) -> torch.Tensor:
        """Copy of a device view as a CPU tensor (synchronises the current stream)."""
        return self.device_view(name, n).cpu()

    def view_ptr(self, name: str) -> int:
        """Raw device address of a state view (e.g. 'psmc_last_tokens')."""
        return getattr(lib(), name)(self._h)

    tokens = property(lambda s: s._view("psmc_tokens", s.R))
    last_tokens = property(lambda s: s._view("psmc_last_tokens", s.R))
    log_weights = property(lambda s: s._view("psmc_log_weights", s.R))
    log_inc = property(lambda s: s._view("psmc_log_inc", s.R))
    logp_tok = property(lambda s: s._view("psmc_logp_tok", s.R))
    cum_logp = property(lambda s: s._view("psmc_cum_logp", s.R))
    ancestors = property(lambda s: s._view("psmc_ancestors", s.R))
    slot_map = property(lambda s: s._view("psmc_slot_map", s.R))
    resampled = property(lambda s: s._view("psmc_resampled", s.G))
    ess = property(lambda s: s._view("psmc_ess", s.G))
    log_z = property(lambda s: s._view("psmc_log_z", s.G))
    lens = property(lambda s: s._view("psmc_lens", s.R))
    mask_sizes = property(lambda s: s._view("psmc_mask_sizes", s.R))
    done = property(lambda s: s._view("psmc_done", s.R))
    move_count = property(lambda s: int(s._view("psmc_move_count", 1)[0]))


def init(N, V, alpha, tau, ess_thresh, ramp, seed, eos_id) -> Psmc:
    """psmc_init: one group."""
    return Psmc(N, V, alpha, tau, ess_thresh, ramp, seed, eos_id)


def init_batched(G, N, V, alpha, tau, ess_thresh, ramp, seed, eos_id, T_max, prompt_len=None) -> Psmc:
    """psmc_init_batched: G independent groups."""
    return Psmc(N, V, alpha, tau, ess_thresh, ramp, seed, eos_id, G=G, T_max=T_max, prompt_len=prompt_len)


def logits_pass_scratch_bytes(R: int, V: int) -> int:
    return lib().psmc_logits_pass_scratch_bytes(R, V)


def step_layout(R: int, V: int, dtype_code: int):
    """psmc_step_layout: (the eight layout words, the CTAs' first granules followed by the total); host only."""
    words = (C.c_int32 * 8)()
    _check(lib().psmc_step_layout(R, V, dtype_code, words, None, 0), "psmc_step_layout")
    shares = (C.c_int32 * (words[1] + 1))()
    _check(lib().psmc_step_layout(R, V, dtype_code, words, shares, len(shares)), "psmc_step_layout")
    return list(words), list(shares)


def step_share_of(R: int, V: int, dtype_code: int, granule: int) -> int:
    return lib().psmc_step_share_of(R, V, dtype_code, granule)


def logits_pass(logits: torch.Tensor, beta: float, alpha_t: float, u: torch.Tensor, done, scratch: torch.Tensor,
                tok: torch.Tensor, logp: torch.Tensor, loginc: torch.Tensor, status_word: torch.Tensor, stream=None):
    """psmc_logits_pass: the stateless logit pass.  All tensors on the GPU; scratch zero-filled uint8."""
    R, V = logits.shape
    assert logits.stride(1) == 1 and u.dtype == torch.float64 and tok.dtype == torch.int32
    _check(lib().psmc_logits_pass(logits.data_ptr(), _dtype_code(logits), R, V, logits.stride(0), beta, alpha_t,
                                  u.data_ptr(), _ptr(done), scratch.data_ptr(), scratch.numel() * scratch.element_size(),
                                  tok.data_ptr(), logp.data_ptr(), loginc.data_ptr(), status_word.data_ptr(),
                                  _stream(stream)), "psmc_logits_pass")


def logits_pass_static(logits: torch.Tensor, beta: float, alpha_t: float, u: torch.Tensor, done, tok: torch.Tensor,
                       logp: torch.Tensor, loginc: torch.Tensor, status_word: torch.Tensor, stream=None):
    """psmc_logits_pass_static: the logit pass without a scratch argument, for callers that cannot allocate.

    The span partials live in a fixed 4 MiB array inside the library; calls share it, so keep them on one
    stream.  Raises PsmcError(E_TOO_LARGE) when logits_pass_scratch_bytes(R, V) exceeds STATIC_SCRATCH_BYTES."""
    R, V = logits.shape
    assert logits.stride(1) == 1 and u.dtype == torch.float64 and tok.dtype == torch.int32
    _check(lib().psmc_logits_pass_static(logits.data_ptr(), _dtype_code(logits), R, V, logits.stride(0), beta,
                                         alpha_t, u.data_ptr(), _ptr(done), tok.data_ptr(), logp.data_ptr(),
                                         loginc.data_ptr(), status_word.data_ptr(), _stream(stream)),
           "psmc_logits_pass_static")
