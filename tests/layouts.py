"""Index maps between the library's physical layouts and plain row-major arrays, written
from the layout description in include/mpfa.h (test helper; numpy only)."""
import numpy as np


def pad128(n):
    return (n + 127) // 128 * 128


def codes_to_logical(codes: np.ndarray, B, H, N) -> np.ndarray:
    """tile-layout codes (flat uint8) -> [B,H,N,64]; also returns the pad rows for a zero check."""
    a = codes.reshape(B, H, pad128(N), 64)
    return a[:, :, :N, :], a[:, :, N:, :]


def sf_to_logical(sf: np.ndarray, B, H, N) -> np.ndarray:
    """tile-layout scale factors (flat uint8) -> [B,H,N_pad,8]."""
    tiles = pad128(N) // 128
    a = sf.reshape(B, H, tiles, 2, 512)
    r = np.arange(128)
    g = np.arange(8)
    off = (r[:, None] % 32) * 16 + (r[:, None] // 32) * 4 + (g[None, :] % 4)     # [128, 8]
    half = np.broadcast_to(g[None, :] // 4, (128, 8))
    out = a[:, :, :, half, off]                                                   # [B,H,tiles,128,8]
    return out.reshape(B, H, tiles * 128, 8)


def paged_k_offset(t, g, j):
    r = t % 8
    return (t // 8) * 512 + r * 64 + ((g // 2) ^ (r // 2)) * 16 + (g % 2) * 8 + j


def paged_v_offset(t, c):
    r = t % 8
    return (t // 8) * 1024 + r * 128 + ((c // 16) ^ r) * 16 + c % 16


def paged_k_to_logical(slab: np.ndarray) -> np.ndarray:
    """[..., 4096] page slab -> [..., 64 tokens, 64 bytes]."""
    t, g, j = np.meshgrid(np.arange(64), np.arange(8), np.arange(8), indexing="ij")
    off = paged_k_offset(t, g, j).reshape(64, 64)
    return slab[..., off]


def paged_v_to_logical(slab: np.ndarray) -> np.ndarray:
    """[..., 8192] page slab -> [..., 64 tokens, 128 channels]."""
    t, c = np.meshgrid(np.arange(64), np.arange(128), indexing="ij")
    return slab[..., paged_v_offset(t, c)]


def paged_delta_to_logical(page: np.ndarray, G: int) -> np.ndarray:
    """[H_q, 64] Delta_S page -> [H_q, 64 tokens]."""
    h = np.arange(page.shape[0])[:, None]
    t = np.arange(64)[None, :]
    return np.take_along_axis(page, (((t // 8) ^ (h % G)) * 8 + t % 8), axis=1)


def v_fp4_to_logical(buf: np.ndarray, B, H, N):
    """FP4 V operand (codes of all tiles, then block scales; flat uint8) -> (codes [B,H,128,NB,8], sf [B,H,128,NB],
    pad codes, pad scales) with NB = ceil(N/16); the pads (blocks past NB) are returned for a zero check."""
    tiles = pad128(N) // 128
    nb = (N + 15) // 16
    n_codes = B * H * tiles * 8192
    c = buf[:n_codes].reshape(B, H, tiles, 128, 8, 8).transpose(0, 1, 3, 2, 4, 5).reshape(B, H, 128, tiles * 8, 8)
    a = buf[n_codes:n_codes + B * H * tiles * 1024].reshape(B, H, tiles, 2, 512)
    ch = np.arange(128)
    kb = np.arange(8)
    off = (ch[:, None] % 32) * 16 + (ch[:, None] // 32) * 4 + (kb[None, :] % 4)      # [128, 8]
    atom = np.broadcast_to(kb[None, :] // 4, (128, 8))
    s = a[:, :, :, atom, off].transpose(0, 1, 3, 2, 4).reshape(B, H, 128, tiles * 8)
    return c[:, :, :, :nb], s[:, :, :, :nb], c[:, :, :, nb:], s[:, :, :, nb:]
