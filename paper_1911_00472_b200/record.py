"""A small convenience wrapper: pinned host copy of a record + the C-ABI handle + torch buffers.

torch is used for memory and streams only (pinned host buffer, device output tensor, the
current stream's handle); all decoding happens behind pcr_decode.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


class Decoder:
    """Opens one record (bytes-like / uint8 numpy array) and decodes it at a chosen fidelity."""

    def __init__(self, record_bytes, device: str | torch.device = "cuda:0", pin: bool = True):
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise RuntimeError("the PCR decoder runs on a CUDA device only")
        arr = np.frombuffer(record_bytes, dtype=np.uint8) if not isinstance(record_bytes, np.ndarray) else record_bytes
        host = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.uint8))
        self.host = host.pin_memory() if pin else host.clone()
        with torch.cuda.device(self.device):
            self.handle = B.pcr_open(self.host.data_ptr(), self.host.numel())
        self.n_images = B.pcr_num_images(self.handle)
        self.n_groups = B.pcr_num_groups(self.handle)
        self.out_bytes = B.pcr_out_bytes(self.handle)
        self.info = [B.pcr_get_image(self.handle, i) for i in range(self.n_images)]
        self.out = None

    def prefix_bytes(self, k: int) -> int:
        return B.pcr_prefix_bytes(self.handle, k)

    def alloc_out(self) -> torch.Tensor:
        return torch.empty(max(self.out_bytes, 16), dtype=torch.uint8, device=self.device)

    def decode(self, k: int, out: torch.Tensor | None = None, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Enqueue the decode at fidelity k on `stream` (default: torch's current stream)."""
        if out is None:
            if self.out is None:
                self.out = self.alloc_out()
            out = self.out
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        with torch.cuda.device(self.device):
            B.pcr_decode(self.handle, k, out.data_ptr(), s.cuda_stream)
        return out

    def decode_more(self, k: int, out: torch.Tensor | None = None, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Raise the fidelity of the last decode to k: only the scans not yet decoded are processed."""
        if out is None:
            if self.out is None:
                self.out = self.alloc_out()
            out = self.out
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        with torch.cuda.device(self.device):
            B.pcr_decode_more(self.handle, k, out.data_ptr(), s.cuda_stream)
        return out

    def decode_tensor(self, k: int, crops: np.ndarray, size: int, mean, std, dtype: torch.dtype = torch.float16,
                      rgb: torch.Tensor | None = None, tensor: torch.Tensor | None = None,
                      stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Decode at fidelity k to a (N, 3, size, size) training batch: crops is an (N, 5) array of
        x0, y0, w, h, flip per image.  Argument marshalling only; the work is pcr_decode_tensor's."""
        crops = np.ascontiguousarray(crops, dtype=np.uint32)
        if crops.shape != (self.n_images, 5):
            raise ValueError("crops must have shape (n_images, 5)")
        codes = {torch.float16: B.PCR_F16, torch.float32: B.PCR_F32, torch.bfloat16: B.PCR_BF16}
        if dtype not in codes:
            raise ValueError("dtype must be torch.float16, torch.bfloat16 or torch.float32")
        m = np.ascontiguousarray(mean, dtype=np.float32)
        sd = np.ascontiguousarray(std, dtype=np.float32)
        if rgb is None:
            if self.out is None:
                self.out = self.alloc_out()
            rgb = self.out
        if tensor is None:
            tensor = torch.empty((self.n_images, 3, size, size), dtype=dtype, device=self.device)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        with torch.cuda.device(self.device):
            B.pcr_decode_tensor(self.handle, k, crops.ctypes.data, size, m.ctypes.data, sd.ctypes.data,
                                codes[dtype], rgb.data_ptr(), tensor.data_ptr(),
                                s.cuda_stream)
        return tensor

    def msssim(self, rgb_a: torch.Tensor, rgb_b: torch.Tensor, stream: torch.cuda.Stream | None = None) -> torch.Tensor:
        """Multi-scale SSIM of every image between two decodes of this record: (N,) float32 on the
        device.  Marshalling only (scratch and result tensors); the work is pcr_msssim's."""
        need = B.pcr_msssim_scratch_bytes(self.handle)
        if getattr(self, "_ms_scratch", None) is None or self._ms_scratch.numel() < need:
            self._ms_scratch = torch.empty(max(need, 16), dtype=torch.uint8, device=self.device)
        scores = torch.empty(self.n_images, dtype=torch.float32, device=self.device)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        with torch.cuda.device(self.device):
            B.pcr_msssim(self.handle, rgb_a.data_ptr(), rgb_b.data_ptr(), self._ms_scratch.data_ptr(), scores.data_ptr(),
                         s.cuda_stream)
        return scores

    def set_upsampling(self, triangle: bool) -> None:
        """Chroma upsampling of later decodes: 2x2 replication (default) or the triangle filter."""
        B.pcr_set_upsampling(self.handle, B.PCR_UPSAMPLE_TRIANGLE if triangle else B.PCR_UPSAMPLE_REPLICATE)

    def evict(self) -> None:
        B.pcr_evict(self.handle)

    def status(self):
        return B.pcr_status(self.handle)

    def image(self, out: torch.Tensor, i: int) -> torch.Tensor:
        """View of image i inside an output buffer: (H, W, 3) uint8."""
        inf = self.info[i]
        return out[inf.out_offset:inf.out_offset + inf.out_bytes].view(inf.height, inf.width, 3)

    def coeffs(self, i: int | None = None) -> torch.Tensor:
        """Coefficient planes of the last decode as a (blocks, 64) int16 device tensor (a copy)."""
        ptr, nbytes = B.pcr_coeffs(self.handle)
        n = nbytes // 2
        iface = {"shape": (n,), "typestr": "<i2", "data": (ptr, False), "version": 2}

        class _Wrap:
            __cuda_array_interface__ = iface

        with torch.cuda.device(self.device):
            t = torch.as_tensor(_Wrap(), device=self.device).view(-1, 64).clone()
        if i is None:
            return t
        a, b = B.pcr_image_blocks(self.handle, i)
        return t[a:a + b]

    def close(self) -> None:
        if getattr(self, "handle", None):
            B.pcr_close(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
