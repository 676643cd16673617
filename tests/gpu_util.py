"""Helpers for the GPU parity tests: move numpy inputs to the device, call the C-ABI through the
binding, bring results back as numpy. No arithmetic of the method lives here."""
import numpy as np
import torch

from paper_2511_11446_b200 import binding as B


def to_dev_bf16(bits_u16: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits_u16.view(np.int16).copy()).cuda().view(torch.bfloat16)


def bf16_to_np(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class DevLayer:
    """Device copy of one layer's constants (weights packed by the library's own host packer)."""

    def __init__(self, w_int8: np.ndarray, s_w: np.ndarray, bias_bits, bits: int):
        self.N, self.K = w_int8.shape
        self.bits = bits
        packed = B.dp_pack_weights_host(np.ascontiguousarray(w_int8), bits)
        self.packed_np = packed
        self.qweight = torch.from_numpy(packed.view(np.uint8).copy()).cuda()
        self.s_w = torch.from_numpy(s_w.copy()).cuda()
        self.bias = None if bias_bits is None else to_dev_bf16(bias_bits)
        self.w = B.make_weight(self.qweight, self.s_w, self.bias, self.N, self.K, bits)


def run_linear(layer: DevLayer, x_bits: np.ndarray, flags=0, taps=True, prequant=None):
    """Returns dict(y, q, s_a, acc, status). prequant = (q int8 np, s_a f32 np) to skip DAQ."""
    M, K = x_bits.shape if prequant is None else prequant[0].shape
    N = layer.N
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.dp_wq_linear_workspace(M, N, K, layer.bits, flags), dtype=torch.uint8, device="cuda")
    dbg = None
    if taps:
        q = torch.full((M, K), 99, dtype=torch.int8, device="cuda")
        s_a = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
        acc = torch.full((M, N), -12345, dtype=torch.int32, device="cuda")
        dbg = B.dp_debug(q.data_ptr(), K, s_a.data_ptr(), acc.data_ptr(), N)
    if prequant is None:
        x = to_dev_bf16(x_bits)
        B.dp_wq_linear(layer.w, x, K, None, M, y, N, ws, dbg, status, flags)
    else:
        xq = torch.from_numpy(prequant[0].copy()).cuda()
        sa = torch.from_numpy(prequant[1].copy()).cuda()
        B.dp_wq_linear(layer.w, xq, K, sa, M, y, N, ws, dbg, status, flags)
    torch.cuda.synchronize()
    out = dict(y=bf16_to_np(y), status=int(status.item()))
    if taps:
        out.update(q=q.cpu().numpy(), s_a=s_a.cpu().numpy(), acc=acc.cpu().numpy())
    return out
