"""Seeded synthetic inputs shaped like the paper's LLaMA decode layers.

Data recipe only: this module holds none of the hot path's arithmetic and is used by the
tests and the benchmark to feed the CUDA library and the CPU checker with the same tensors.
All draws come from a torch.Generator seeded from (base seed, tensor id), on the requested
device; a given (seed, device type) always yields the same tensors.

  LUT          [N][4] fp16: four draws from N(0, 0.02^2), rounded to fp16, then sorted ascending.
               Group-wise variant [N][K/G][4]: the same, drawn independently for every group of
               G weights of a row (G = 128, the paper's weight group size).
  codes        uniform on {0,1,2,3}, or: w ~ Laplace(0, b=0.02), each row rotated along K by the
               same normalized block-Hadamard as the layer's activations (stand-in for the
               offline weight rotation of Section 4.1), then mapped to the nearest of the
               row's four levels (ties to the lower index).
  activations  [M][K] fp16: N(0,1), each element independently multiplied by 20 with probability 0.01.
"""
import math

import torch


def _gen(seed: int, tensor_id: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(tensor_id) * 7919) % (2 ** 63 - 1))
    return g


def make_lut(N: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, 1, device)
    lv = torch.randn(N, 4, generator=g, device=device, dtype=torch.float64) * 0.02
    lv = lv.to(torch.float16)
    lv, _ = torch.sort(lv, dim=1)
    return lv.contiguous()


def make_lut_grouped(N: int, NG: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, 5, device)
    lv = torch.randn(N, NG, 4, generator=g, device=device, dtype=torch.float64) * 0.02
    lv = lv.to(torch.float16)
    lv, _ = torch.sort(lv, dim=2)
    return lv.contiguous()


def make_codes_uniform(N: int, K: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, 2, device)
    return torch.randint(0, 4, (N, K), generator=g, device=device, dtype=torch.uint8)


def _block_rotate_rows_f64(w: torch.Tensor, B: int) -> torch.Tensor:
    """Rows of w (float64 [R][K]) times blockdiag(H_B): butterflies on a reshaped view."""
    if B <= 1:
        return w
    R, K = w.shape
    v = w.reshape(R, K // B, B)
    h = 1
    while h < B:
        v = v.reshape(R, K // B, B // (2 * h), 2, h)
        a = v[:, :, :, 0, :]
        b = v[:, :, :, 1, :]
        v = torch.stack((a + b, a - b), dim=3)
        h *= 2
    return (v.reshape(R, K) / math.sqrt(B))


def make_codes_rotated_laplace(N: int, K: int, had_block: int, lut: torch.Tensor, seed: int,
                               device="cpu", max_chunk_elems: int = 1 << 26) -> torch.Tensor:
    g = _gen(seed, 3, device)
    out = torch.empty(N, K, dtype=torch.uint8, device=device)
    rows = max(1, min(N, max_chunk_elems // K))
    lut64 = lut.to(device=device, dtype=torch.float64)
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        u = torch.rand(r1 - r0, K, generator=g, device=device, dtype=torch.float64) - 0.5
        w = -0.02 * torch.sign(u) * torch.log1p(-2.0 * u.abs())
        w = _block_rotate_rows_f64(w, had_block)
        lv = lut64[r0:r1]
        if lv.dim() == 3:   # group-wise grid [rows][K/G][4]: every weight sees its group's levels
            lv = lv.repeat_interleave(K // lv.shape[1], dim=1).permute(0, 2, 1)   # [rows][4][K]
        else:
            lv = lv[:, :, None]                                                  # [rows][4][1]
        best = torch.zeros(r1 - r0, K, dtype=torch.uint8, device=device)
        bestd = (w - lv[:, 0]).abs()
        for c in (1, 2, 3):
            d = (w - lv[:, c]).abs()
            better = d < bestd  # strict: ties keep the lower index
            best = torch.where(better, torch.full_like(best, c), best)
            bestd = torch.where(better, d, bestd)
        out[r0:r1] = best
    return out


def make_layer_grouped(N: int, K: int, G: int, had_block: int, codes_kind: str, seed: int, device="cpu"):
    """Returns (codes u8 [N][K], lut fp16 [N][K/G][4])."""
    lut = make_lut_grouped(N, K // G, seed, device)
    if codes_kind == "uniform":
        codes = make_codes_uniform(N, K, seed, device)
    elif codes_kind == "rotated_laplace":
        codes = make_codes_rotated_laplace(N, K, had_block, lut, seed, device, max_chunk_elems=1 << 24)
    else:
        raise ValueError(codes_kind)
    return codes, lut


def make_activations(M: int, K: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, 4, device)
    x = torch.randn(M, K, generator=g, device=device, dtype=torch.float32)
    hit = torch.rand(M, K, generator=g, device=device) < 0.01
    x = torch.where(hit, x * 20.0, x)
    return x.to(torch.float16).contiguous()


def make_layer(N: int, K: int, had_block: int, codes_kind: str, seed: int, device="cpu"):
    """Returns (codes u8 [N][K], lut fp16 [N][4])."""
    lut = make_lut(N, seed, device)
    if codes_kind == "uniform":
        codes = make_codes_uniform(N, K, seed, device)
    elif codes_kind == "rotated_laplace":
        codes = make_codes_rotated_laplace(N, K, had_block, lut, seed, device)
    else:
        raise ValueError(codes_kind)
    return codes, lut
