"""Helpers for the GPU parity tests: call the C ABI on torch-owned device memory."""
from __future__ import annotations

import numpy as np
import torch

from paper_1705_01626_b200 import binding as B

DT = {torch.float32: B.F32, torch.float16: B.F16, torch.bfloat16: B.BF16, torch.uint8: B.U8}
NP_RAW = {4: np.uint32, 2: np.uint16, 1: np.uint8}
TORCH_RAW = {4: torch.int32, 2: torch.int16, 1: torch.uint8}
CANARY = 0xA7


def raw_numpy(x: torch.Tensor) -> np.ndarray:
    """Host copy of a tensor's bit patterns as a flat unsigned array."""
    flat = x.detach().contiguous().view(-1)
    return flat.view(TORCH_RAW[x.element_size()]).cpu().numpy().view(NP_RAW[x.element_size()])


class DeviceCodec:
    """Buffers for one compress/decompress of up to n elements, with canaries
    behind the payload capacity and the table."""

    def __init__(self, n: int, dtype: torch.dtype, capacity: int | None = None, device="cuda"):
        self.n, self.dtype, self.code = n, dtype, DT[dtype]
        self.s = torch.empty(0, dtype=dtype).element_size()
        self.cap = B.cdma_zvc_max_compressed_bytes(n, self.code) if capacity is None else capacity
        self.entries = B.cdma_zvc_table_entries(n)
        self.ws_bytes = B.cdma_zvc_workspace_bytes(n, self.code)
        self.guard = 256
        self.payload = torch.full((self.cap + self.guard,), CANARY, dtype=torch.uint8, device=device)
        self.table = torch.full((self.entries + 4,), -0x5A5A5A5A5A5A5A5B, dtype=torch.int64, device=device)
        # workspace deliberately dirty: the library must not depend on its contents
        self.ws = torch.full((self.ws_bytes,), 0xFF, dtype=torch.uint8, device=device)

    def compress(self, x: torch.Tensor, layout=B.NCHW, stream=0) -> int:
        assert x.is_contiguous() and x.numel() == self.n
        return B.cdma_zvc_compress(x.data_ptr() if self.n else 0, self.n, self.code, layout,
                                   self.payload.data_ptr(), self.cap, self.table.data_ptr(),
                                   self.ws.data_ptr(), self.ws_bytes, stream)

    def decompress(self, out: torch.Tensor, src_bytes: int, layout=B.NCHW, stream=0) -> int:
        return B.cdma_zvc_decompress(self.payload.data_ptr(), src_bytes, self.table.data_ptr(), self.n,
                                     self.code, layout, out.data_ptr() if self.n else 0,
                                     self.ws.data_ptr(), self.ws_bytes, stream)

    def payload_numpy(self, c: int) -> np.ndarray:
        return self.payload[:c].cpu().numpy()

    def table_numpy(self) -> np.ndarray:
        return self.table[: self.entries].cpu().numpy().view(np.uint64)

    def canaries_intact(self) -> bool:
        tail = self.payload[self.cap:].cpu().numpy()
        ttail = self.table[self.entries:].cpu().numpy()
        return bool((tail == CANARY).all() and (ttail == -0x5A5A5A5A5A5A5A5B).all())

    def load(self, payload: np.ndarray, table: np.ndarray):
        """Put a (possibly doctored) stream and table on the device."""
        self.payload[: len(payload)] = torch.from_numpy(np.ascontiguousarray(payload)).cuda()
        self.table[: len(table)] = torch.from_numpy(np.ascontiguousarray(table).view(np.int64)).cuda()
