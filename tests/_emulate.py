"""A CPU emulation of an fp32 data path for the Gated MLP, for the tests only.

It is neither the oracle (fp64, the plain definition) nor the product: it computes what a faithful
fp32-accumulating implementation computes - bf16 inputs, fp32 products and sums, one rounding of H to bf16, fp32
down projection, one rounding of Y - so that a test can say how many elements ANY such implementation leaves
beyond a tolerance that the fp64 oracle defines.  The K reduction runs in chunks (a library fp32 matmul inside a
chunk, sequential fp32 additions between chunks), the structure of the GPU kernels' accumulation chains.
"""
import numpy as np
import torch


def _bf16_bits_to_f32(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy((bits.astype(np.uint32) << 16).view(np.float32))


def fp32_path_rows(X, Wg, Wu, Wd, rows, chunk: int = 512, col_block: int = 4096):
    """(y, h) for the given rows: y float64 array of the bf16-rounded outputs, h float64 array of the bf16 H."""
    x = _bf16_bits_to_f32(np.ascontiguousarray(X[rows]))
    K, N = Wg.shape
    h = torch.empty(x.shape[0], N, dtype=torch.float32)
    for n0 in range(0, N, col_block):
        g = torch.zeros(x.shape[0], min(col_block, N - n0), dtype=torch.float32)
        u = torch.zeros_like(g)
        for k0 in range(0, K, chunk):
            xs = x[:, k0:k0 + chunk]
            g += xs @ _bf16_bits_to_f32(np.ascontiguousarray(Wg[k0:k0 + chunk, n0:n0 + col_block]))
            u += xs @ _bf16_bits_to_f32(np.ascontiguousarray(Wu[k0:k0 + chunk, n0:n0 + col_block]))
        h[:, n0:n0 + col_block] = ((g / (1.0 + torch.exp(-g))) * u).to(torch.bfloat16).to(torch.float32)
    y = torch.zeros(x.shape[0], Wd.shape[1], dtype=torch.float32)
    for k0 in range(0, N, chunk):
        y += h[:, k0:k0 + chunk] @ _bf16_bits_to_f32(np.ascontiguousarray(Wd[k0:k0 + chunk]))
    return y.to(torch.bfloat16).to(torch.float64).numpy(), h.to(torch.float64).numpy()
