"""Algorithm 1 of DIVISION on top of torch.autograd: activation maps that autograd would keep for the backward pass
are cached as (H^L, V^H, Delta, delta) instead (forward loop: pooling, residual, Quant, cache) and rebuilt when
the backward pass asks for them (backward loop: Dequant, up-sample and add, free).

Glue only: every step of the pair runs in the CUDA library through the C ABI; torch owns the buffers and the
graph.  `DivisionCache` installs saved-tensor hooks; `DivisionReLU` / `DivisionDropout` are the paper's appendix
operators that cache a packed 1-bit mask instead of an activation map.

    model = to_division_modules(model)            # nn.ReLU / nn.Dropout -> mask-caching operators
    with DivisionCache(block=8, qbits=2) as cache:
        loss = model(x).sum()
    loss.backward()                               # saved maps are decompressed as the backward pass reaches them
    print(cache.raw_bytes / cache.cached_bytes)

What is compressed: CUDA tensors of dtype fp32 / bf16 with 3 or 4 dimensions (Minibatch x Channel x N and
Minibatch x Channel x N x N) and at least `min_elems` elements that are not leaves requiring grad (parameters).
Everything else autograd saves is kept as it is.  All calls go to the current stream.  Every compress call gets a
scratch slice of its own (a few KB, from an arena that is reused from one forward pass to the next), so calls on
different streams do not meet in it, and its device-side status word stays readable: the first decompress of a
backward pass (or `check()`) reads all of them back in one copy and raises if a bounded wait inside a compress
kernel ran out, instead of handing a corrupt activation map to the backward pass.
"""
from __future__ import annotations

import weakref

import torch

from . import binding

_DTYPES = {torch.float32: "f32", torch.bfloat16: "bf16"}


class _Cached:
    """What replaces one saved activation map: the blob and what is needed to rebuild the tensor."""
    __slots__ = ("blob", "codec_key", "shape", "dtype", "planegroup")

    def __init__(self, blob, codec_key, shape, dtype, planegroup):
        self.blob, self.codec_key, self.shape, self.dtype, self.planegroup = blob, codec_key, shape, dtype, planegroup


def should_compress(shape, dtype, is_cuda: bool, is_param_like: bool, min_elems: int) -> bool:
    """The selection rule stated in the module docstring (pure function of tensor metadata)."""
    if not is_cuda or dtype not in _DTYPES or is_param_like:
        return False
    if len(shape) not in (3, 4):
        return False
    n = 1
    for s in shape:
        n *= int(s)
    return n >= min_elems and min(int(s) for s in shape) >= 1


class DivisionCache:
    """Context manager: inside it, activation maps saved for backward are cached in compressed form."""

    def __init__(self, block: int = 8, qbits: int = 2, lfc_dtype: str | None = None, seed: int = 0,
                 min_elems: int = 1 << 14, per_plane: bool = False):
        self.block, self.qbits, self.lfc_dtype, self.seed = int(block), int(qbits), lfc_dtype, int(seed)
        self.min_elems, self.per_plane = int(min_elems), bool(per_plane)
        self.raw_bytes = 0          # bytes autograd would have kept for the maps that were compressed
        self.cached_bytes = 0       # bytes of their blobs (closed form)
        self.maps = 0
        self.records = []           # (seed, shape, dtype name) per compressed map, in forward order
        self._descs = {}
        self._arena = []            # [tensor, bytes used] scratch chunks; a compress call takes a slice of its own
        self._slices = []           # (chunk index, byte offset) of the slices handed out since __enter__
        self._checked = 0           # slices whose status word has been read back
        self._seen = {}
        self._hooks = None

    # -- descriptors and scratch ------------------------------------------------------------------------------
    def _descriptor(self, shape4, dtype_name):
        key = (shape4, dtype_name)
        if key not in self._descs:
            lfc = self.lfc_dtype or dtype_name
            desc = binding.make_desc(*shape4, self.block, self.qbits, dtype_name, lfc)
            layout = binding.div_planegroup_bytes(desc) if self.per_plane else binding.div_compressed_bytes(desc)
            self._descs[key] = (desc, layout)
        return key, self._descs[key]

    ARENA_CHUNK_BYTES = 1 << 20

    def _scratch(self, nbytes, device):
        """A scratch slice of its own for one compress call (256-byte aligned, never shared with another call)."""
        need = (int(nbytes) + 255) // 256 * 256
        for ci, entry in enumerate(self._arena):
            chunk, used = entry
            if chunk.device == device and used + need <= chunk.numel():
                entry[1] = used + need
                self._slices.append((ci, used))
                return chunk[used:used + need]
        chunk = torch.empty(max(self.ARENA_CHUNK_BYTES, need), dtype=torch.uint8, device=device)
        self._arena.append([chunk, need])
        self._slices.append((len(self._arena) - 1, 0))
        return chunk[:need]

    def check(self):
        """Read back the device-side status words of the compress calls made since the last check (one gather per
        arena chunk, host-blocking) and raise DivisionError if a bounded wait ran out in one of them."""
        todo = self._slices[self._checked:]
        self._checked = len(self._slices)
        by_chunk = {}
        for ci, off in todo:
            by_chunk.setdefault(ci, []).append(off // 4)
        for ci, words in by_chunk.items():
            chunk = self._arena[ci][0]
            idx = torch.tensor(words, dtype=torch.int64).to(chunk.device, non_blocking=True)
            status = chunk.view(torch.int32).index_select(0, idx).cpu()
            bad = status.nonzero()
            if bad.numel():
                raise binding.DivisionError(int(status[bad[0, 0]]), "div_compress (device side, seen by DivisionCache)")

    # -- hooks ------------------------------------------------------------------------------------------------
    def pack(self, t: torch.Tensor):
        is_param_like = t.requires_grad and t.is_leaf
        if not should_compress(tuple(t.shape), t.dtype, t.is_cuda, is_param_like, self.min_elems) or not t.is_contiguous():
            return t
        # the same map saved by two operators (a convolution and the shortcut convolution of a residual block):
        # recognised only while the first tensor object is still alive, so a reused address cannot be mistaken for it
        hit = self._seen.get(id(t))
        if hit is not None and hit[0]() is t and hit[1] == t._version:
            return hit[2]
        shape = tuple(t.shape)
        shape4 = shape if len(shape) == 4 else (shape[0], shape[1], 1, shape[2])
        name = _DTYPES[t.dtype]
        key, (desc, layout) = self._descriptor(shape4, name)
        blob = torch.empty(int(layout.total_bytes), dtype=torch.uint8, device=t.device)
        seed = self.seed + self.maps
        stream = binding.current_stream_handle()
        if self.per_plane:
            binding.div_planegroup_compress(desc, t.data_ptr(), blob.data_ptr(), blob.numel(), seed, stream)
        else:
            ws = self._scratch(layout.workspace_bytes, t.device)
            binding.div_compress(desc, t.data_ptr(), blob.data_ptr(), blob.numel(), ws.data_ptr(), ws.numel(), seed, stream)
        self.maps += 1
        self.raw_bytes += int(layout.raw_bytes)
        self.cached_bytes += int(layout.closed_form_bytes)
        self.records.append((seed, shape, name))
        handle = _Cached(blob, key, shape, t.dtype, self.per_plane)
        self._seen[id(t)] = (weakref.ref(t), t._version, handle)
        return handle

    def unpack(self, h):
        if not isinstance(h, _Cached):
            return h
        if self._checked < len(self._slices):
            self.check()
        desc, _ = self._descs[h.codec_key]
        out = torch.empty(h.shape, dtype=h.dtype, device=h.blob.device)
        stream = binding.current_stream_handle()
        if h.planegroup:
            binding.div_planegroup_decompress(desc, h.blob.data_ptr(), h.blob.numel(), out.data_ptr(), stream)
        else:
            binding.div_decompress(desc, h.blob.data_ptr(), h.blob.numel(), out.data_ptr(), stream)
        return out

    def __enter__(self):
        # the arena is reused: what the previous forward pass put there has been consumed by its kernels, which
        # precede this pass's kernels on the stream
        for entry in self._arena:
            entry[1] = 0
        self._slices = []
        self._checked = 0
        self._hooks = torch.autograd.graph.saved_tensors_hooks(self.pack, self.unpack)
        self._hooks.__enter__()
        return self

    def __exit__(self, *exc):
        self._seen = {}                  # identities are only meaningful during the forward pass
        return self._hooks.__exit__(*exc)


# ------------------------------------------------------------------------------------------------------------
# mask-caching operators (appendix algorithms "Relu operator" and "Dropout operator")
# ------------------------------------------------------------------------------------------------------------
class _MaskFunction(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, drop_threshold, seed):
        if not (x.is_cuda and x.dtype in _DTYPES):
            raise ValueError("the mask operators run on CUDA tensors of dtype float32 or bfloat16")
        x = x.contiguous()
        total = x.numel()
        y = torch.empty_like(x)
        nbytes = binding.div_mask_bytes(total)
        mask = torch.empty(nbytes, dtype=torch.uint8, device=x.device)
        name = _DTYPES[x.dtype]
        stream = binding.current_stream_handle()
        if drop_threshold is None:
            binding.div_relu_forward(x.data_ptr(), y.data_ptr(), mask.data_ptr(), nbytes, total, name, stream)
        else:
            binding.div_dropout_forward(x.data_ptr(), y.data_ptr(), mask.data_ptr(), nbytes, total, seed, drop_threshold,
                                        name, stream)
        ctx.mask, ctx.total, ctx.name = mask, total, name      # the packed mask is all that is cached
        return y

    @staticmethod
    def backward(ctx, g):
        g = g.contiguous()
        gin = torch.empty_like(g)
        binding.div_mask_backward(ctx.mask.data_ptr(), ctx.mask.numel(), g.data_ptr(), gin.data_ptr(), ctx.total, ctx.name,
                                  binding.current_stream_handle())
        return gin, None, None


class DivisionReLU(torch.nn.Module):
    """ReLU that caches one bit per element for its backward pass."""

    def forward(self, x):
        return _MaskFunction.apply(x, None, 0)


class DivisionDropout(torch.nn.Module):
    """Dropout as printed in the paper's appendix (kept values are not rescaled); caches one bit per element."""

    def __init__(self, p: float = 0.5, seed: int = 0):
        super().__init__()
        self.drop_threshold = int(round(float(p) * 65536))
        if not 0 <= self.drop_threshold <= 65536:
            raise ValueError("p must lie in [0, 1]")
        self.seed, self.calls = int(seed), 0

    def forward(self, x):
        if not self.training:
            return x
        self.calls += 1
        return _MaskFunction.apply(x, self.drop_threshold, self.seed + self.calls)


def to_division_modules(module: torch.nn.Module) -> torch.nn.Module:
    """Replace every nn.ReLU in `module` by DivisionReLU (in place; returns the module)."""
    for name, child in list(module.named_children()):
        if isinstance(child, torch.nn.ReLU):
            setattr(module, name, DivisionReLU())
        else:
            to_division_modules(child)
    return module
