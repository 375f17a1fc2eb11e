"""ctypes binding of the C ABI (argument marshalling only).  PyTorch provides device memory and
streams; nothing here computes."""
from __future__ import annotations
import ctypes as C
import os
import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libeas_encoder.so")
_lib = None

STATUS_NAMES = {0: "EAS_OK", 1: "EAS_ERR_INVALID_ARG", 2: "EAS_ERR_UNSUPPORTED", 3: "EAS_ERR_WORKSPACE",
                4: "EAS_ERR_CUDA", 5: "EAS_ERR_DEVICE_TIMEOUT", 6: "EAS_ERR_ARCH", 7: "EAS_ERR_DEVICE_CHECK"}

EXPORTED_SYMBOLS = [
    "eas_encoder_create", "eas_encoder_weight_arena_bytes", "eas_encoder_workspace_bytes", "eas_encoder_out_rows",
    "eas_encode_microbatch", "eas_encode_microbatch_static", "eas_encoder_status", "eas_encoder_last_launch_count", "eas_encoder_set_attention_impl",
    "eas_encoder_set_graph_mode", "eas_encoder_graph_stats", "eas_encoder_enable_timing", "eas_encoder_timing_read", "eas_last_error", "eas_encoder_destroy", "eas_kernel_gemm", "eas_kernel_gemm_tile", "eas_kernel_norm", "eas_kernel_attention",
    "eas_encoder_set_split_k", "eas_encoder_set_norm_fold", "eas_sm_partition_create", "eas_sm_partition_sm_count", "eas_sm_partition_stream", "eas_sm_partition_destroy",
]


class EasError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {text}")
        self.status = status


class ArchConfig(C.Structure):
    _fields_ = [("family", C.c_int32), ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("d_mlp", C.c_int32), ("norm", C.c_int32), ("norm_eps", C.c_float), ("mlp", C.c_int32),
                ("in_channels", C.c_int32), ("patch", C.c_int32), ("temporal_patch", C.c_int32),
                ("has_cls", C.c_int32), ("embed_norm", C.c_int32), ("final_norm", C.c_int32), ("pos", C.c_int32),
                ("max_pos", C.c_int32), ("rope_theta", C.c_float), ("head", C.c_int32),
                ("d_head_hidden", C.c_int32), ("d_out", C.c_int32), ("out_dtype", C.c_int32)]


class Tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dev_ptr", C.c_void_p), ("ndim", C.c_int32), ("shape", C.c_int64 * 4)]


class Weights(C.Structure):
    _fields_ = [("tensors", C.POINTER(Tensor)), ("n_tensors", C.c_int32), ("arena", C.c_void_p),
                ("arena_bytes", C.c_size_t)]


class PackedInputs(C.Structure):
    _fields_ = [("data", C.c_void_p), ("n_items", C.c_int32), ("item_shape", C.POINTER(C.c_int32)),
                ("item_offset", C.POINTER(C.c_int64)), ("cu_seqlens_host", C.POINTER(C.c_int32)),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


def load_library():
    """dlopen the built library and declare the signatures.  Raises if it is missing: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_31551_b200.build` "
                           "(the encoder has no CPU or PyTorch fallback)")
    lib = C.CDLL(_LIB_PATH)
    lib.eas_encoder_create.restype = C.c_int
    lib.eas_encoder_create.argtypes = [C.POINTER(ArchConfig), C.POINTER(Weights), C.POINTER(C.c_void_p)]
    lib.eas_encoder_weight_arena_bytes.restype = C.c_size_t
    lib.eas_encoder_weight_arena_bytes.argtypes = [C.POINTER(ArchConfig)]
    lib.eas_encoder_workspace_bytes.restype = C.c_size_t
    lib.eas_encoder_workspace_bytes.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32]
    lib.eas_encoder_out_rows.restype = C.c_int64
    lib.eas_encoder_out_rows.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_int32]
    lib.eas_encode_microbatch.restype = C.c_int
    lib.eas_encode_microbatch.argtypes = [C.c_void_p, C.POINTER(PackedInputs), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    lib.eas_encode_microbatch_static.restype = C.c_int
    lib.eas_encode_microbatch_static.argtypes = [C.c_void_p, C.POINTER(PackedInputs), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    lib.eas_encoder_status.restype = C.c_int
    lib.eas_encoder_status.argtypes = [C.c_void_p, C.c_void_p]
    lib.eas_encoder_last_launch_count.restype = C.c_int32
    lib.eas_encoder_last_launch_count.argtypes = [C.c_void_p]
    lib.eas_encoder_set_attention_impl.restype = C.c_int
    lib.eas_encoder_set_attention_impl.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_encoder_set_split_k.restype = C.c_int
    lib.eas_encoder_set_split_k.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_encoder_set_norm_fold.restype = C.c_int
    lib.eas_encoder_set_norm_fold.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_encoder_set_graph_mode.restype = C.c_int
    lib.eas_encoder_set_graph_mode.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_encoder_graph_stats.restype = C.c_int
    lib.eas_encoder_graph_stats.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
    lib.eas_encoder_enable_timing.restype = C.c_int
    lib.eas_encoder_enable_timing.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_encoder_timing_read.restype = C.c_int32
    lib.eas_encoder_timing_read.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_float)]
    lib.eas_last_error.restype = C.c_char_p
    lib.eas_last_error.argtypes = []
    lib.eas_encoder_destroy.restype = None
    lib.eas_encoder_destroy.argtypes = [C.c_void_p]
    lib.eas_kernel_gemm.restype = C.c_int
    lib.eas_kernel_gemm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                    C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.eas_kernel_gemm_tile.restype = C.c_int
    lib.eas_kernel_gemm_tile.argtypes = lib.eas_kernel_gemm.argtypes + [C.c_int32]
    lib.eas_kernel_norm.restype = C.c_int
    lib.eas_kernel_norm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                    C.c_float, C.c_int32, C.c_int32, C.c_void_p]
    lib.eas_kernel_attention.restype = C.c_int
    lib.eas_kernel_attention.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32), C.c_int32, C.c_int32, C.c_int32,
                                         C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
    lib.eas_sm_partition_create.restype = C.c_int
    lib.eas_sm_partition_create.argtypes = [C.c_int32, C.POINTER(C.c_void_p)]
    lib.eas_sm_partition_sm_count.restype = C.c_int32
    lib.eas_sm_partition_sm_count.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_sm_partition_stream.restype = C.c_void_p
    lib.eas_sm_partition_stream.argtypes = [C.c_void_p, C.c_int32]
    lib.eas_sm_partition_destroy.restype = None
    lib.eas_sm_partition_destroy.argtypes = [C.c_void_p]
    _lib = lib
    return lib


def _check(status: int):
    if status != 0:
        raise EasError(status, load_library().eas_last_error().decode())


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def arch_struct(cfg: dict) -> ArchConfig:
    a = ArchConfig()
    for name, _ in ArchConfig._fields_:
        setattr(a, name, cfg.get("out_dtype", 0) if name == "out_dtype" else cfg[name])
    return a


def weights_to_device(weights: dict, device="cuda") -> dict:
    """name -> bf16 device tensor, from float32 arrays that hold bf16-exact values (lossless cast)."""
    return {k: torch.from_numpy(np.ascontiguousarray(v)).to(device=device, dtype=torch.bfloat16).contiguous()
            for k, v in weights.items()}


def pack_items(items, device="cuda"):
    """Concatenate items (arrays of bf16-exact float32 values) back to back, each starting on a 16-byte
    boundary.  Returns (device bf16 buffer, item offsets in elements)."""
    offsets, total = [], 0
    for it in items:
        offsets.append(total)
        total += (it.size + 7) // 8 * 8
    host = torch.zeros(total, dtype=torch.bfloat16, pin_memory=torch.cuda.is_available())
    for it, off in zip(items, offsets):
        host[off:off + it.size] = torch.from_numpy(np.ascontiguousarray(it).reshape(-1)).to(torch.bfloat16)
    return host.to(device, non_blocking=True), offsets


class Encoder:
    """Handle of eas_encoder_create.  Keeps the weight tensors and the arena alive."""

    def __init__(self, cfg: dict, dev_weights: dict):
        self.lib = load_library()
        self.cfg = dict(cfg)
        self._arch = arch_struct(cfg)
        self._weights = dev_weights
        names = list(dev_weights.keys())
        self._name_bytes = [n.encode() for n in names]
        arr = (Tensor * len(names))()
        for i, n in enumerate(names):
            t = dev_weights[n]
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous(), n
            arr[i].name = self._name_bytes[i]
            arr[i].dev_ptr = t.data_ptr()
            arr[i].ndim = t.dim()
            for j, s in enumerate(t.shape):
                arr[i].shape[j] = s
        self._tensor_arr = arr
        arena_bytes = self.lib.eas_encoder_weight_arena_bytes(C.byref(self._arch))
        if arena_bytes == 0:
            raise EasError(1, self.lib.eas_last_error().decode())
        self._arena = torch.empty(arena_bytes, dtype=torch.uint8, device="cuda")
        w = Weights(arr, len(names), self._arena.data_ptr(), arena_bytes)
        handle = C.c_void_p()
        _check(self.lib.eas_encoder_create(C.byref(self._arch), C.byref(w), C.byref(handle)))
        self.handle = handle
        self._workspace = None

    def close(self):
        if getattr(self, "handle", None):
            self.lib.eas_encoder_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace_bytes(self, total_tokens: int, n_items: int, max_seqlen: int = 0) -> int:
        return self.lib.eas_encoder_workspace_bytes(self.handle, total_tokens, n_items, max_seqlen)

    def out_rows(self, cu_seqlens_host) -> int:
        cu = np.ascontiguousarray(cu_seqlens_host, dtype=np.int32)
        return self.lib.eas_encoder_out_rows(self.handle, cu.ctypes.data_as(C.POINTER(C.c_int32)), len(cu) - 1)

    def set_attention_impl(self, impl: int):
        _check(self.lib.eas_encoder_set_attention_impl(self.handle, impl))

    def encode_microbatch(self, data: torch.Tensor, item_shapes, item_offsets, cu_seqlens_host,
                          cu_seqlens_dev: torch.Tensor | None = None, sm_budget: int = 0, stream=None,
                          out: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
        """eas_encode_microbatch.  data: device bf16 buffer; item_shapes [(frames,h,w)]; item_offsets in
        elements; cu_seqlens_host: int32 [n+1].  Returns the device bf16 [out_rows, d_out] tensor (enqueued,
        not synchronised)."""
        n = len(item_shapes)
        shp = np.ascontiguousarray(item_shapes, dtype=np.int32).reshape(n, 3)
        offs = np.ascontiguousarray(item_offsets, dtype=np.int64)
        cu = np.ascontiguousarray(cu_seqlens_host, dtype=np.int32)
        if cu_seqlens_dev is None:
            cu_seqlens_dev = torch.from_numpy(cu).to(data.device)
        T = int(cu[-1])
        need = self.workspace_bytes(T, n)
        if workspace is None:
            if self._workspace is None or self._workspace.numel() < need + 1024:
                self._workspace = torch.empty(need + 1024, dtype=torch.uint8, device=data.device)
            workspace = self._workspace
        # the library wants a 1024-byte aligned workspace; small torch allocations are only 512-byte aligned
        ws_ptr = (workspace.data_ptr() + 1023) // 1024 * 1024
        ws_bytes = workspace.numel() - (ws_ptr - workspace.data_ptr())
        if out is None:
            rows = self.out_rows(cu)
            out = torch.empty((max(rows, 0), self.cfg["d_out"]), device=data.device,
                              dtype=torch.float32 if self.cfg.get("out_dtype", 0) else torch.bfloat16)
        pin = PackedInputs(data.data_ptr(), n, shp.ctypes.data_as(C.POINTER(C.c_int32)),
                           offs.ctypes.data_as(C.POINTER(C.c_int64)), cu.ctypes.data_as(C.POINTER(C.c_int32)),
                           ws_ptr, ws_bytes)
        _check(self.lib.eas_encode_microbatch(self.handle, C.byref(pin), cu_seqlens_dev.data_ptr(), sm_budget,
                                              _stream_ptr(stream), out.data_ptr()))
        self._keep = (cu_seqlens_dev, workspace)
        return out

    def encode_microbatch_static(self, data: torch.Tensor, item_shapes, item_offsets, cu_seqlens_host,
                                 cu_seqlens_dev: torch.Tensor, out: torch.Tensor, sm_budget: int = 0, stream=None):
        """eas_encode_microbatch_static: the forward pass on the scratch built into the library.  Nothing is
        allocated here either: the caller passes the device cu_seqlens and the output tensor."""
        n = len(item_shapes)
        shp = np.ascontiguousarray(item_shapes, dtype=np.int32).reshape(n, 3)
        offs = np.ascontiguousarray(item_offsets, dtype=np.int64)
        cu = np.ascontiguousarray(cu_seqlens_host, dtype=np.int32)
        pin = PackedInputs(data.data_ptr(), n, shp.ctypes.data_as(C.POINTER(C.c_int32)),
                           offs.ctypes.data_as(C.POINTER(C.c_int64)), cu.ctypes.data_as(C.POINTER(C.c_int32)), None, 0)
        _check(self.lib.eas_encode_microbatch_static(self.handle, C.byref(pin), cu_seqlens_dev.data_ptr(), sm_budget,
                                                     _stream_ptr(stream), out.data_ptr()))
        return out

    def set_split_k(self, on: bool):
        """eas_encoder_set_split_k: small micro-batches split the K loop of the residual GEMMs (default off)."""
        _check(self.lib.eas_encoder_set_split_k(self.handle, 1 if on else 0))

    def set_norm_fold(self, on: bool):
        """eas_encoder_set_norm_fold: the blocks' normalisations inside the GEMMs around them (default off)."""
        _check(self.lib.eas_encoder_set_norm_fold(self.handle, 1 if on else 0))

    def set_graph_mode(self, on: bool):
        """eas_encoder_set_graph_mode: replay captured forward passes for repeated micro-batch shapes.  Needs a
        non-default stream, and the same data / cu_seqlens_dev / out / workspace tensors from call to call."""
        _check(self.lib.eas_encoder_set_graph_mode(self.handle, int(on)))

    def graph_stats(self) -> dict:
        h, c, n = C.c_int64(0), C.c_int64(0), C.c_int32(0)
        _check(self.lib.eas_encoder_graph_stats(self.handle, C.byref(h), C.byref(c), C.byref(n)))
        return {"hits": h.value, "captures": c.value, "cached": n.value}

    def status(self, stream=None):
        """eas_encoder_status: synchronises the stream and raises on a device-side error."""
        _check(self.lib.eas_encoder_status(self.handle, _stream_ptr(stream)))

    def enable_timing(self, on: bool):
        _check(self.lib.eas_encoder_enable_timing(self.handle, int(on)))

    def timing_read(self):
        """-> (kernel classes int32 [n], milliseconds float32 [n]) of the last timed call, in launch order."""
        n = self.lib.eas_encoder_timing_read(self.handle, 0, None, None)
        cls = np.zeros(max(n, 1), dtype=np.int32)
        ms = np.zeros(max(n, 1), dtype=np.float32)
        got = self.lib.eas_encoder_timing_read(self.handle, n, cls.ctypes.data_as(C.POINTER(C.c_int32)),
                                               ms.ctypes.data_as(C.POINTER(C.c_float)))
        if got < 0:
            raise EasError(4, "timing read failed")
        return cls[:got], ms[:got]

    def last_launch_count(self) -> int:
        return self.lib.eas_encoder_last_launch_count(self.handle)


class SmPartition:
    """eas_sm_partition: the device's SMs split into side 0 (the encoder, at least `sm_encode` SMs) and side 1 (the
    neighbour, the rest), one stream on each (Section 3.4).  `stream(side)` is a torch stream object over the
    library's stream; the handle owns it, so keep this object alive while the streams are in use."""

    def __init__(self, sm_encode: int):
        self.lib = load_library()
        h = C.c_void_p()
        _check(self.lib.eas_sm_partition_create(int(sm_encode), C.byref(h)))
        self.handle = h
        self._streams = [torch.cuda.ExternalStream(self.lib.eas_sm_partition_stream(h, s)) for s in (0, 1)]

    def sm_count(self, side: int) -> int:
        return self.lib.eas_sm_partition_sm_count(self.handle, side)

    def stream(self, side: int):
        return self._streams[side]

    def close(self):
        if self.handle is not None:
            self.lib.eas_sm_partition_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def kernel_gemm(A, W, bias, act=0, out_fp32=False, resid=None, sm_budget=0, stream=None, out=None, status=None,
                tile_shape=0):
    """eas_kernel_gemm (eas_kernel_gemm_tile when tile_shape != 0) on device tensors.  Returns (out, device status
    word).  `status` (device int32, zeroed by the caller) can be passed in so that a call allocates nothing."""
    lib = load_library()
    M, K = A.shape
    N = W.shape[0]
    if out is None:
        out = torch.empty((M, N // 2 if act == 2 else N), dtype=torch.float32 if out_fp32 else torch.bfloat16, device=A.device)
    if status is None:
        status = torch.zeros(4, dtype=torch.int32, device=A.device)
    args = (A.data_ptr(), W.data_ptr(), bias.data_ptr(), out.data_ptr(),
            resid.data_ptr() if resid is not None else None, M, N, K, act, int(out_fp32), sm_budget,
            _stream_ptr(stream), status.data_ptr())
    if tile_shape:
        _check(lib.eas_kernel_gemm_tile(*args, tile_shape))
    else:
        _check(lib.eas_kernel_gemm(*args))
    return out, status


def kernel_norm(x, gamma, beta, kind, eps, out_fp32=False, sm_budget=0, stream=None):
    lib = load_library()
    rows, d = x.shape
    y = torch.empty((rows, d), dtype=torch.float32 if out_fp32 else torch.bfloat16, device=x.device)
    _check(lib.eas_kernel_norm(x.data_ptr(), y.data_ptr(), gamma.data_ptr() if gamma is not None else None,
                               beta.data_ptr() if beta is not None else None, rows, d, kind, eps, int(out_fp32),
                               sm_budget, _stream_ptr(stream)))
    return y


def kernel_attention(qkv, cu_seqlens_host, n_heads, head_dim, sm_budget=0, stream=None, impl=0):
    lib = load_library()
    cu = np.ascontiguousarray(cu_seqlens_host, dtype=np.int32)
    T = qkv.shape[0]
    out = torch.empty((T, n_heads * head_dim), dtype=torch.bfloat16, device=qkv.device)
    status = torch.zeros(4, dtype=torch.int32, device=qkv.device)
    _check(lib.eas_kernel_attention(qkv.data_ptr(), out.data_ptr(), cu.ctypes.data_as(C.POINTER(C.c_int32)), len(cu) - 1,
                                    n_heads, head_dim, sm_budget, _stream_ptr(stream), impl, status.data_ptr()))
    return out, status
