"""Thin binding of liblgc (include/lgc.h): same names, argument marshalling only.

PyTorch provides device memory and the stream; every step of the path runs in the library's
CUDA kernels.  There is no fallback: if the library cannot be loaded, or no CUDA device is
present, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblgc.so")

LGC_OK = 0
VARIANT_RAR, VARIANT_PS = 0, 1
AE_CONV2, AE_IDENTITY, AE_CONV5 = 0, 1, 2
LAYER_TOPK_AE, LAYER_TOPK_ONLY, LAYER_DENSE = 0, 1, 2
LAYER_MODES = {"ae": LAYER_TOPK_AE, "topk": LAYER_TOPK_ONLY, "dense": LAYER_DENSE}

EXPORTS = (
    "lgc_workspace_bytes", "lgc_init", "lgc_destroy", "lgc_accumulate", "lgc_topk", "lgc_encode",
    "lgc_combine", "lgc_decode_scatter", "lgc_topk_scatter", "lgc_abort_step", "lgc_ae_train_step", "lgc_ae_train_step_ps",
    "lgc_encode_indices", "lgc_encode_innovation_positions", "lgc_dense_mean", "lgc_step_host",
    "lgc_get_layout", "lgc_keep_counts", "lgc_get_slots", "lgc_get_buffers", "lgc_set_ae_params", "lgc_get_ae_params",
    "lgc_check", "lgc_status_string", "lgc_last_error", "lgc_topk_noalloc", "lgc_topk_noalloc_check", "lgc_kernel_launches",
    "lgc_selection_stats",
)
NOALLOC_MAX_N = 16777216


class lgc_config(C.Structure):
    _fields_ = [
        ("num_nodes", C.c_int32), ("num_layers", C.c_int32), ("layer_numel", C.POINTER(C.c_int64)),
        ("density_ppm", C.c_uint32), ("innovation_permille", C.c_uint32), ("momentum", C.c_float),
        ("variant", C.c_int32), ("ae_kind", C.c_int32), ("ae_c1", C.c_int32), ("ae_c2", C.c_int32),
        ("adam_lr", C.c_float), ("adam_beta1", C.c_float), ("adam_beta2", C.c_float), ("adam_eps", C.c_float),
        ("stream", C.c_void_p), ("grad_row_stride", C.c_int64), ("layer_mode", C.POINTER(C.c_uint8)),
    ]


_lib = None


def lib() -> C.CDLL:
    """Loads liblgc.so; raises if it has not been built (``python -m paper_2103_08870_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2103_08870_b200.build`")
        l = C.CDLL(LIB_PATH)
        vp, sz = C.c_void_p, C.c_size_t
        l.lgc_workspace_bytes.argtypes = [C.POINTER(lgc_config), C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
        l.lgc_init.argtypes = [C.POINTER(lgc_config), vp, sz, vp, sz, vp, sz, C.POINTER(vp)]
        l.lgc_destroy.argtypes = [vp]
        l.lgc_accumulate.argtypes = [vp, vp, C.c_int32]
        l.lgc_topk.argtypes = [vp, C.c_int32, vp]
        l.lgc_encode.argtypes = [vp]
        l.lgc_combine.argtypes = [vp, C.c_int32]
        l.lgc_decode_scatter.argtypes = [vp, vp]
        l.lgc_topk_scatter.argtypes = [vp, vp]
        l.lgc_abort_step.argtypes = [vp]
        l.lgc_ae_train_step.argtypes = [vp, vp]
        l.lgc_ae_train_step_ps.argtypes = [vp, C.c_int32, C.c_float, C.c_float, vp]
        l.lgc_encode_indices.argtypes = [vp, C.c_int32, vp, C.c_size_t, vp]
        l.lgc_encode_innovation_positions.argtypes = [vp, C.c_int32, vp, C.c_size_t, vp]
        l.lgc_dense_mean.argtypes = [vp, C.c_int64, C.c_int32, C.c_int64, vp, vp]
        l.lgc_step_host.argtypes = [vp, vp, vp, vp, vp, C.c_int32]
        l.lgc_get_layout.argtypes = [vp] + [C.POINTER(C.c_int64)] * 5
        l.lgc_keep_counts.argtypes = [vp]
        l.lgc_keep_counts.restype = C.POINTER(C.c_int64)
        l.lgc_get_buffers.argtypes = [vp] + [C.POINTER(vp)] * 8
        l.lgc_get_slots.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.POINTER(C.c_int64)), C.POINTER(vp)]
        l.lgc_set_ae_params.argtypes = [vp, vp, sz]
        l.lgc_get_ae_params.argtypes = [vp, vp, sz]
        l.lgc_check.argtypes = [vp]
        l.lgc_status_string.argtypes = [C.c_int]
        l.lgc_status_string.restype = C.c_char_p
        l.lgc_last_error.argtypes = [vp]
        l.lgc_last_error.restype = C.c_char_p
        l.lgc_topk_noalloc.argtypes = [vp, C.c_int64, C.c_int64, vp, vp]
        l.lgc_topk_noalloc_check.argtypes = [vp]
        l.lgc_selection_stats.argtypes = [vp] + [C.POINTER(C.c_int64)] * 5
        l.lgc_kernel_launches.argtypes = []
        l.lgc_kernel_launches.restype = C.c_uint64
        for name in EXPORTS:            # every declared entry point must be exported
            getattr(l, name)
        _lib = l
    return _lib


class LGCError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        name = lib().lgc_status_string(status).decode()
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail else ""))


def dense_mean(grads: torch.Tensor, update: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """update[j] = node-ordered mean over the K rows of `grads` ([K][n] fp32 CUDA view, unit column stride)."""
    if not (grads.is_cuda and grads.dtype == torch.float32 and grads.dim() == 2 and grads.stride(1) == 1):
        raise ValueError("grads: need a 2-D fp32 CUDA view with unit column stride")
    K, n = grads.shape
    if not (update.is_cuda and update.dtype == torch.float32 and update.is_contiguous() and update.numel() == n):
        raise ValueError(f"update: need a contiguous fp32 CUDA tensor of {n} elements")
    st = stream if stream is not None else torch.cuda.current_stream(grads.device)
    status = lib().lgc_dense_mean(grads.data_ptr(), grads.stride(0) if K > 1 else n, K, n, update.data_ptr(),
                                  C.c_void_p(st.cuda_stream))
    if status != LGC_OK:
        raise LGCError(status, "lgc_dense_mean", lib().lgc_last_error(None).decode())


def topk_noalloc(v: torch.Tensor, k: int, idx_out: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """lgc_topk_noalloc: indices of the k largest |v| of one flat fp32 CUDA vector, with the work
    space inside the library (for callers that cannot allocate or pass scratch).  At most
    NOALLOC_MAX_N elements; calls must not overlap on the GPU (they share the work space)."""
    if not (v.is_cuda and v.dtype == torch.float32 and v.is_contiguous() and v.dim() == 1):
        raise ValueError("v: need a contiguous 1-D fp32 CUDA tensor")
    if not (idx_out.is_cuda and idx_out.dtype == torch.int32 and idx_out.is_contiguous() and idx_out.numel() == k):
        raise ValueError("idx_out: need a contiguous int32 CUDA tensor of k elements")
    s = stream if stream is not None else torch.cuda.current_stream(v.device)
    st = lib().lgc_topk_noalloc(v.data_ptr(), v.numel(), k, idx_out.data_ptr(), C.c_void_p(s.cuda_stream))
    if st != LGC_OK:
        raise LGCError(st, "lgc_topk_noalloc", lib().lgc_last_error(None).decode())


def topk_noalloc_check(stream: Optional[torch.cuda.Stream] = None) -> None:
    """lgc_topk_noalloc_check: waits for the stream and raises if a kernel of lgc_topk_noalloc recorded an inconsistency."""
    s = stream if stream is not None else torch.cuda.current_stream()
    st = lib().lgc_topk_noalloc_check(C.c_void_p(s.cuda_stream))
    if st != LGC_OK:
        raise LGCError(st, "lgc_topk_noalloc_check", lib().lgc_last_error(None).decode())


def kernel_launches() -> int:
    """Kernels the library has enqueued from this thread so far."""
    return int(lib().lgc_kernel_launches())


def status_string(status: int) -> str:
    return lib().lgc_status_string(status).decode()


class LGC:
    """One LGC context and the device buffers it works in.

    Methods are the C entry points without the ``lgc_`` prefix; tensors are passed as device
    pointers.  Views of the library's buffers are exposed as torch tensors (no copies).
    """

    def __init__(self, layer_numel: Sequence[int], num_nodes: int, density_ppm: int = 1000,
                 momentum: float = 0.9, variant: str = "rar", ae_kind: str = "conv2", c1: int = 8,
                 c2: int = 4, innovation_permille: int = 100, lr: float = 0.0, beta1: float = 0.0,
                 beta2: float = 0.0, eps: float = 0.0, device: Optional[torch.device] = None,
                 stream: Optional[torch.cuda.Stream] = None, grad_row_stride: int = 0,
                 layer_mode: Optional[Sequence] = None):
        """layer_mode: per layer "ae" / "topk" / "dense" (or the lgc_layer_mode numbers); None = every layer "ae"."""
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2103_08870_b200.lgc needs a CUDA device; there is no CPU path")
        self._l = lib()
        self.device = torch.device(device if device is not None else "cuda:0")
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._numel = (C.c_int64 * len(layer_numel))(*[int(n) for n in layer_numel])
        self._modes = None
        if layer_mode is not None:
            if len(layer_mode) != len(layer_numel):
                raise ValueError("layer_mode: one entry per layer")
            self._modes = (C.c_uint8 * len(layer_numel))(*[LAYER_MODES.get(m, m) for m in layer_mode])
        self.cfg = lgc_config(
            num_nodes=num_nodes, num_layers=len(layer_numel), layer_numel=self._numel,
            density_ppm=density_ppm, innovation_permille=innovation_permille, momentum=momentum,
            variant={"rar": VARIANT_RAR, "ps": VARIANT_PS}[variant],
            ae_kind={"conv2": AE_CONV2, "identity": AE_IDENTITY, "conv5": AE_CONV5}[ae_kind], ae_c1=c1, ae_c2=c2,
            adam_lr=lr, adam_beta1=beta1, adam_beta2=beta2, adam_eps=eps,
            stream=C.c_void_p(self.stream.cuda_stream), grad_row_stride=grad_row_stride,
            layer_mode=self._modes if self._modes is not None else C.POINTER(C.c_uint8)())
        self.grad_row_stride = grad_row_stride
        self.variant, self.ae_kind, self.K, self.c1, self.c2 = variant, ae_kind, num_nodes, c1, c2
        sb, wb, pb = C.c_size_t(), C.c_size_t(), C.c_size_t()
        self._ctx = C.c_void_p()
        self._ok(self._l.lgc_workspace_bytes(C.byref(self.cfg), C.byref(sb), C.byref(wb), C.byref(pb)),
                 "lgc_workspace_bytes")
        self.state_bytes, self.scratch_bytes, self.params_bytes = sb.value, wb.value, pb.value
        self.state = torch.empty(sb.value, dtype=torch.uint8, device=self.device)
        self.scratch = torch.empty(wb.value, dtype=torch.uint8, device=self.device)
        self.params_buf = torch.zeros(pb.value // 4, dtype=torch.float32, device=self.device)
        self._ok(self._l.lgc_init(C.byref(self.cfg), self.state.data_ptr(), sb.value, self.scratch.data_ptr(),
                                  wb.value, self.params_buf.data_ptr(), pb.value, C.byref(self._ctx)), "lgc_init")
        vals = [C.c_int64() for _ in range(5)]
        self._ok(self._l.lgc_get_layout(self._ctx, *[C.byref(v) for v in vals]), "lgc_get_layout")
        self.N, self.mu, self.L1, self.L2, self.P = (v.value for v in vals)
        self.L = len(layer_numel)
        kc = self._l.lgc_keep_counts(self._ctx)
        self.k_l = [kc[i] for i in range(self.L)]
        mu_all, slots, vt = C.c_int64(), C.POINTER(C.c_int64)(), C.c_void_p()
        self._ok(self._l.lgc_get_slots(self._ctx, C.byref(mu_all), C.byref(slots), C.byref(vt)), "lgc_get_slots")
        self.mu_all, self.mu_t = mu_all.value, mu_all.value - self.mu
        self.first_slot = [slots[i] for i in range(self.L)]      # of each layer's kept entries in a row of idx; -1: dense
        self._val_t_ptr = vt.value
        self.S = self.K if variant == "ps" else 1
        self.code_len = self.mu if ae_kind == "identity" else c2 * self.L2
        if ae_kind == "conv5":          # four stride-2 convolutions, four code channels, stored [L4][4]
            n = self.mu
            for _ in range(4):
                n = (n - 3) // 2 + 1
            self.L4, self.code_len = n, 4 * n

    # -- plumbing -----------------------------------------------------------------------------
    def _ok(self, status: int, where: str) -> None:
        if status != LGC_OK:
            detail = self._l.lgc_last_error(self._ctx if self._ctx else None).decode()
            raise LGCError(status, where, detail)

    def close(self) -> None:
        if self._ctx:
            self._l.lgc_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _dev_f32(t: torch.Tensor, numel: int, name: str) -> int:
        if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.numel() == numel):
            raise ValueError(f"{name}: need a contiguous fp32 CUDA tensor of {numel} elements")
        return t.data_ptr()

    # -- the stages ---------------------------------------------------------------------------
    def accumulate(self, grads: torch.Tensor, leader_hint: int = -1) -> None:
        """grads: fp32 CUDA, K x N; with a grad_row_stride a [K][N] view whose rows are that far apart."""
        if self.grad_row_stride:
            if not (grads.is_cuda and grads.dtype == torch.float32 and tuple(grads.shape) == (self.K, self.N)
                    and grads.stride(1) == 1 and (self.K == 1 or grads.stride(0) == self.grad_row_stride)):
                raise ValueError("grads: need a [K][N] fp32 CUDA view with unit column stride and the configured row stride")
            ptr = grads.data_ptr()
        else:
            ptr = self._dev_f32(grads, self.K * self.N, "grads")
        self._ok(self._l.lgc_accumulate(self._ctx, ptr, leader_hint), "lgc_accumulate")

    def topk(self, leader: int = 0, update_hint: Optional[torch.Tensor] = None) -> None:
        ptr = self._dev_f32(update_hint, self.N, "update_hint") if update_hint is not None else None
        self._ok(self._l.lgc_topk(self._ctx, leader, ptr), "lgc_topk")

    def encode(self) -> None:
        self._ok(self._l.lgc_encode(self._ctx), "lgc_encode")

    def combine(self, common_node: int = 0) -> None:
        self._ok(self._l.lgc_combine(self._ctx, common_node), "lgc_combine")

    def decode_scatter(self, update: torch.Tensor) -> None:
        self._ok(self._l.lgc_decode_scatter(self._ctx, self._dev_f32(update, self.N, "update")), "lgc_decode_scatter")

    def topk_scatter(self, update: torch.Tensor) -> None:
        self._ok(self._l.lgc_topk_scatter(self._ctx, self._dev_f32(update, self.N, "update")), "lgc_topk_scatter")

    def abort_step(self) -> None:
        self._ok(self._l.lgc_abort_step(self._ctx), "lgc_abort_step")

    def ae_train_step(self, loss_out: Optional[torch.Tensor] = None) -> None:
        ptr = self._dev_f32(loss_out, 1, "loss_out") if loss_out is not None else None
        self._ok(self._l.lgc_ae_train_step(self._ctx, ptr), "lgc_ae_train_step")

    def ae_train_step_ps(self, common_node: int, lambda_rec: float = 1.0, lambda_sim: float = 1.0,
                         loss_out: Optional[torch.Tensor] = None) -> None:
        ptr = self._dev_f32(loss_out, 1, "loss_out") if loss_out is not None else None
        self._ok(self._l.lgc_ae_train_step_ps(self._ctx, common_node, lambda_rec, lambda_sim, ptr), "lgc_ae_train_step_ps")

    def encode_indices(self, node: int, stream_out: torch.Tensor, sizes_out: torch.Tensor) -> None:
        """DEFLATE stream of `node`'s index list into `stream_out` (uint8, CUDA, a multiple of 4 bytes);
        `sizes_out` (int64[2], CUDA) gets the stream's and the varint form's byte counts."""
        if not (stream_out.is_cuda and stream_out.dtype == torch.uint8 and stream_out.is_contiguous()):
            raise ValueError("stream_out: need a contiguous uint8 CUDA tensor")
        if not (sizes_out.is_cuda and sizes_out.dtype == torch.int64 and sizes_out.numel() == 2):
            raise ValueError("sizes_out: need an int64 CUDA tensor of 2 elements")
        self._ok(self._l.lgc_encode_indices(self._ctx, node, stream_out.data_ptr(), stream_out.numel(), sizes_out.data_ptr()),
                 "lgc_encode_indices")

    def encode_innovation_positions(self, node: int, stream_out: torch.Tensor, sizes_out: torch.Tensor) -> None:
        """The same for the positions of `node`'s innovation (parameter server; between combine and decode_scatter)."""
        if not (stream_out.is_cuda and stream_out.dtype == torch.uint8 and stream_out.is_contiguous()):
            raise ValueError("stream_out: need a contiguous uint8 CUDA tensor")
        if not (sizes_out.is_cuda and sizes_out.dtype == torch.int64 and sizes_out.numel() == 2):
            raise ValueError("sizes_out: need an int64 CUDA tensor of 2 elements")
        self._ok(self._l.lgc_encode_innovation_positions(self._ctx, node, stream_out.data_ptr(), stream_out.numel(),
                                                         sizes_out.data_ptr()), "lgc_encode_innovation_positions")

    def step(self, grads: torch.Tensor, update: torch.Tensor, choice: int = 0) -> None:
        """The five stages of one compression step, in order."""
        self.accumulate(grads, choice)
        self.topk(choice, update)
        self.encode()
        self.combine(choice)
        self.decode_scatter(update)

    def step_host(self, host_grads: torch.Tensor, dev_grads: torch.Tensor, dev_update: torch.Tensor,
                  host_update: torch.Tensor, choice: int = 0) -> None:
        for t, n, name in ((host_grads, self.K * self.N, "host_grads"), (host_update, self.N, "host_update")):
            if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous() or t.numel() != n:
                raise ValueError(f"{name}: need a contiguous fp32 host tensor of {n} elements")
        self._ok(self._l.lgc_step_host(self._ctx, host_grads.data_ptr(),
                                       self._dev_f32(dev_grads, self.K * self.N, "dev_grads"),
                                       self._dev_f32(dev_update, self.N, "dev_update"),
                                       host_update.data_ptr(), choice), "lgc_step_host")

    def selection_stats(self):
        """(large (row, layer) pairs, pairs served by the last accumulate, candidates in total, largest
        count, pairs finished from the data)."""
        v = [C.c_int64() for _ in range(5)]
        self._ok(self._l.lgc_selection_stats(self._ctx, *[C.byref(x) for x in v]), "lgc_selection_stats")
        return tuple(x.value for x in v)

    def check(self) -> None:
        self._ok(self._l.lgc_check(self._ctx), "lgc_check")

    # -- parameters ---------------------------------------------------------------------------
    def set_ae_params(self, p: torch.Tensor) -> None:
        p = p.detach().to(torch.float32).contiguous()
        self._keep = p
        self._ok(self._l.lgc_set_ae_params(self._ctx, p.data_ptr(), p.numel()), "lgc_set_ae_params")

    def get_ae_params(self) -> torch.Tensor:
        out = torch.empty(self.P, dtype=torch.float32)
        self._ok(self._l.lgc_get_ae_params(self._ctx, out.data_ptr(), out.numel()), "lgc_get_ae_params")
        return out

    # -- views of the library's buffers ---------------------------------------------------------
    def _buffers(self):
        ptrs = [C.c_void_p() for _ in range(8)]
        self._ok(self._l.lgc_get_buffers(self._ctx, *[C.byref(p) for p in ptrs]), "lgc_get_buffers")
        return [p.value for p in ptrs]

    def _view(self, owner: torch.Tensor, ptr: Optional[int], shape, dtype) -> Optional[torch.Tensor]:
        if not ptr:
            return None
        off = ptr - owner.data_ptr()
        n = 1
        for s in shape:
            n *= s
        size = n * torch.empty((), dtype=dtype).element_size()
        assert 0 <= off and off + size <= owner.numel() * owner.element_size()
        return owner.view(torch.uint8)[off:off + size].view(dtype).view(*shape)

    @property
    def u(self) -> torch.Tensor:
        return self._view(self.state, self._buffers()[0], (self.K, self.N), torch.float32)

    @property
    def v(self) -> torch.Tensor:
        return self._view(self.state, self._buffers()[1], (self.K, self.N), torch.float32)

    @property
    def idx(self) -> torch.Tensor:
        return self._view(self.scratch, self._buffers()[2], (self.S, self.mu_all), torch.int32)

    @property
    def val(self) -> torch.Tensor:
        return self._view(self.scratch, self._buffers()[3], (self.K, self.mu), torch.float32)

    @property
    def val_topk_only(self) -> Optional[torch.Tensor]:
        return self._view(self.scratch, self._val_t_ptr, (self.K, self.mu_t), torch.float32)

    @property
    def code(self) -> torch.Tensor:
        return self._view(self.scratch, self._buffers()[4], (self.K, self.code_len), torch.float32)

    @property
    def combined(self) -> torch.Tensor:
        return self._view(self.scratch, self._buffers()[5], (self.code_len,), torch.float32)

    @property
    def inn(self) -> Optional[torch.Tensor]:
        return self._view(self.scratch, self._buffers()[6], (self.K, self.mu), torch.float32)

    @property
    def recon(self) -> torch.Tensor:
        return self._view(self.scratch, self._buffers()[7], (self.S, self.mu), torch.float32)
