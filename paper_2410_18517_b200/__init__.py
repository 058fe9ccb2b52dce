"""Decode attention over a layer-shared KV cache (KVSharer's inference path) for B200.

``binding`` exposes the C ABI one to one.  ``SharedKVCache`` is a small holder
that lets PyTorch own the device memory (pool and workspace tensors) and the
stream, and forwards every operation to the compiled library.
"""
from __future__ import annotations

from . import binding
from .binding import (  # noqa: F401
    KVS_BF16, KVS_F32, KVS_OK, KVS_OPT_EARLY_START, KVS_OPT_FINISH_IN_KERNEL, KVS_OPT_HOST_CHUNKS, KVS_OPT_KERNEL, KVS_OPT_MAX_CTAS, KVS_OPT_REPLAY, KVS_OPT_WAIT_LIMIT_US, KvsError,
)

__all__ = ["binding", "SharedKVCache", "KvsError"]


class SharedKVCache:
    """One context + the torch tensors backing it.

    ``share_map[l] == l``: layer l computes its own K/V; ``share_map[l] == s < l``:
    layer l reads layer s's cache and appends nothing.
    """

    def __init__(self, n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_seq, dtype="bf16",
                 share_map=None, softmax_scale=0.0, device=0):
        import torch

        self._torch = torch
        self.device = torch.device("cuda", device)
        self.dtype = {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]
        self.shape = (n_layers, n_q_heads, n_kv_heads, head_dim)
        self.max_batch = max_batch
        self.ctx = binding.kvs_create(n_layers, n_q_heads, n_kv_heads, head_dim, max_batch, max_seq,
                                      KVS_BF16 if dtype == "bf16" else KVS_F32, softmax_scale, device)
        try:
            if share_map is not None:
                binding.kvs_set_share_map(self.ctx, share_map)
            self.pool_bytes, self.workspace_bytes = binding.kvs_required_bytes(self.ctx)
            self.pool = self._allocate(self.pool_bytes)
            self.workspace = self._allocate(self.workspace_bytes)
            binding.kvs_bind_memory(self.ctx, self.pool, self.pool_bytes, self.workspace, self.workspace_bytes)
        except Exception:
            binding.kvs_destroy(self.ctx)
            self.ctx = None
            raise

    def _allocate(self, nbytes):
        """Device memory for the pool or the workspace (256-byte aligned uint8 tensor of ``nbytes``)."""
        return self._torch.empty(nbytes, dtype=self._torch.uint8, device=self.device)

    def close(self):
        if getattr(self, "ctx", None):
            self._torch.cuda.synchronize(self.device)
            binding.kvs_destroy(self.ctx)
            self.ctx = None
            self.pool = self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream(self) -> int:
        return self._torch.cuda.current_stream(self.device).cuda_stream

    def append(self, layer, k=None, v=None, batch=None, n_new=None):
        """k, v: ``[batch][n_new][n_kv_heads][head_dim]`` contiguous device tensors (None on a sharing layer)."""
        if k is not None:
            assert k.is_contiguous() and v.is_contiguous() and k.dtype == self.dtype and v.dtype == self.dtype
            assert k.shape == v.shape and k.shape[2:] == (self.shape[2], self.shape[3])
            batch, n_new = k.shape[0], k.shape[1]
        binding.kvs_append(self.ctx, layer, k, v, batch, n_new, self._stream())

    def decode_attention(self, layer, q, out=None):
        """q: ``[batch][n_q_heads][head_dim]``; returns float32 ``[batch][n_q_heads][head_dim]``."""
        torch = self._torch
        assert q.is_contiguous() and q.dtype == self.dtype and q.shape[1:] == (self.shape[1], self.shape[3])
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=self.device)
        binding.kvs_decode_attention(self.ctx, layer, q, out, q.shape[0], self._stream())
        return out

    def decode_step(self, layer, q, k=None, v=None, out=None):
        """Append one token's k, v (``[batch][1][n_kv_heads][head_dim]``; None on a sharing layer) and attend
        with q: ``append`` then ``decode_attention`` in one call, the append riding in the attention kernel."""
        torch = self._torch
        assert q.is_contiguous() and q.dtype == self.dtype and q.shape[1:] == (self.shape[1], self.shape[3])
        if k is not None:
            assert k.is_contiguous() and v.is_contiguous() and k.dtype == self.dtype and v.dtype == self.dtype
            assert k.shape == v.shape == (q.shape[0], 1, self.shape[2], self.shape[3])
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=self.device)
        binding.kvs_decode_step(self.ctx, layer, q, k, v, out, q.shape[0], self._stream())
        return out

    def prefill_attention(self, layer, q, out=None):
        """q: ``[batch][n_q][n_q_heads][head_dim]`` (the newest n_q positions, causal); returns float32 of that shape."""
        torch = self._torch
        assert q.is_contiguous() and q.dtype == self.dtype and q.ndim == 4
        assert q.shape[2:] == (self.shape[1], self.shape[3])
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32, device=self.device)
        binding.kvs_prefill_attention(self.ctx, layer, q, out, q.shape[0], q.shape[1], self._stream())
        return out

    def evict(self, layer, keep, n_keep):
        """keep: device int32 ``[batch][Hkv][stride]`` ascending row lists; n_keep: ``[batch][Hkv]`` counts (host)."""
        assert keep.is_contiguous() and keep.dtype == self._torch.int32 and keep.ndim == 3
        counts = [int(x) for x in self._torch.as_tensor(n_keep).reshape(-1).tolist()]
        binding.kvs_evict(self.ctx, layer, keep, counts, keep.shape[2], keep.shape[0], self._stream())

    def unit_len(self, layer, b, h):
        return binding.kvs_unit_len(self.ctx, layer, b, h)

    def layer_distances(self, batch=None):
        """float32 ``[L][L]`` distances between the layers' sample-mean K/V representations."""
        torch = self._torch
        L = self.shape[0]
        dist = torch.empty(L, L, dtype=torch.float32, device=self.device)
        if batch is None:
            batch = self._cached_batch()
        binding.kvs_layer_distances(self.ctx, batch, dist, self._stream())
        return dist

    def _cached_batch(self):
        b = 0
        while b < self.max_batch and self.unit_len(0, b, 0) > 0:
            b += 1
        return b

    def mean_cosine(self, a, b):
        """cos(mean over samples of a, mean over samples of b) for ``[S][dim]`` device tensors (float32 scalar tensor)."""
        torch = self._torch
        assert a.shape == b.shape and a.ndim == 2 and a.is_contiguous() and b.is_contiguous() and a.dtype == self.dtype
        out = torch.empty(1, dtype=torch.float32, device=self.device)
        binding.kvs_mean_cosine(self.ctx, a, b, a.shape[0], a.shape[1], out, self._stream())
        return out

    def replay_advance(self):
        binding.kvs_replay_advance(self.ctx, self._stream())

    def replay_commit(self, times_run):
        binding.kvs_replay_commit(self.ctx, times_run, self._stream())

    def step_host(self, q_host, k_host, v_host, out_host):
        """One decode step over all layers from host tensors (see ``kvs_step_host``)."""
        return binding.kvs_step_host(self.ctx, q_host, k_host, v_host, out_host, q_host.shape[1], self._stream())

    def plane(self, slot, kv):
        """View of plane (slot, kv) as ``[max_batch][n_kv_heads][row_stride][head_dim]``."""
        off = binding.kvs_plane_offset(self.ctx, slot, kv)
        nxt = binding.kvs_plane_offset(self.ctx, 0, 1)
        rs = binding.kvs_row_stride(self.ctx)
        return self.pool[off:off + nxt].view(self.dtype).view(-1, self.shape[2], rs, self.shape[3])

    # plain forwards
    def num_slots(self):
        return binding.kvs_num_slots(self.ctx)

    def slot_of_layer(self, layer):
        return binding.kvs_slot_of_layer(self.ctx, layer)

    def seq_len(self, layer):
        return binding.kvs_seq_len(self.ctx, layer)

    def reset(self):
        binding.kvs_reset(self.ctx)

    def truncate(self, n_tokens):
        """Cut every slot back to at most ``n_tokens`` rows (host bookkeeping only)."""
        binding.kvs_truncate(self.ctx, n_tokens)

    def clear_device_status(self):
        binding.kvs_clear_device_status(self.ctx, self._stream())

    def selftest_wait_timeout(self, limit_us=1000):
        """Make one bounded device-side wait run out; returns the nanoseconds it lasted."""
        return binding.kvs_selftest_wait_timeout(self.ctx, limit_us, self._stream())

    def stats(self):
        return binding.kvs_stats(self.ctx)

    def device_status(self):
        return binding.kvs_last_device_status(self.ctx)

    def set_option(self, option, value):
        binding.kvs_set_option(self.ctx, option, value)

    def last_launch(self):
        return binding.kvs_last_launch(self.ctx)
