"""Helpers shared by the tests: bit-pattern conversions and oracle <-> device marshalling."""
import numpy as np
import torch

from oracle import qp_oracle as orc


def bits_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 / fp16 tensor -> numpy uint16 bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_from_f32(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def bf16_val(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def cache_to_packed(cache, desc=None) -> orc.Packed:
    """Device cache (binding's Cache) -> oracle Packed with numpy arrays (copies to host).  Only the
    n_keep tokens in use are taken (the arrays may have room for more); `desc` overrides the cache's
    own descriptor when another copy of it has been advanced by appends."""
    d = desc if desc is not None else cache.desc
    n, g = d.n_keep, d.group
    if d.bits == 16:
        return orc.Packed(16, g, n, np.ascontiguousarray(bits_u16(cache.k_codes)[:, :, :n]),
                          np.ascontiguousarray(bits_u16(cache.v_codes)[:, :, :n]), None, None, None, None)
    u32 = lambda t, m: np.ascontiguousarray(t.detach().cpu().contiguous().numpy().view(np.uint32)[:, :, :m])
    h16 = lambda t, m: np.ascontiguousarray(bits_u16(t)[:, :, :m])
    return orc.Packed(d.bits, g, n, u32(cache.k_codes, n // g), u32(cache.v_codes, n),
                      h16(cache.k_scale, n // g), h16(cache.k_zero, n // g),
                      h16(cache.v_scale, n), h16(cache.v_zero, n))


def assert_packed_equal(got: orc.Packed, ref: orc.Packed) -> None:
    assert got.bits == ref.bits and got.n == ref.n
    assert np.array_equal(got.k_codes, ref.k_codes), "k_codes differ"
    assert np.array_equal(got.v_codes, ref.v_codes), "v_codes differ"
    if ref.bits < 16:
        assert np.array_equal(got.k_scale, ref.k_scale), "k_scale differ"
        assert np.array_equal(got.k_zero, ref.k_zero), "k_zero differ"
        assert np.array_equal(got.v_scale, ref.v_scale), "v_scale differ"
        assert np.array_equal(got.v_zero, ref.v_zero), "v_zero differ"


def check_kept_against_oracle(kept_gpu: np.ndarray, pooled_ref: np.ndarray, L: int, w: int, n: int,
                              rel: float = 1e-5) -> int:
    """Index parity with the near-tie rule: the GPU set may differ from the oracle's only in
    positions whose oracle score lies within `rel` (relative) of the oracle's k-th score.
    Returns the number of tolerated swaps.  Structure (ascending, unique, window last) is exact."""
    P, k = L - w, n - w
    ref = orc.select(pooled_ref, L, w, n)
    swaps = 0
    Bt, Hkv, _ = kept_gpu.shape
    for b in range(Bt):
        for h in range(Hkv):
            g, r = kept_gpu[b, h], ref[b, h]
            assert np.all(np.diff(g) > 0), "kept indices not strictly ascending"
            assert g[k:].tolist() == list(range(P, L)), "window tokens not kept last"
            assert g.min() >= 0 and g.max() < L
            if np.array_equal(g, r):
                continue
            s = pooled_ref[b, h]
            kth = np.sort(s)[::-1][k - 1]
            only_g = np.setdiff1d(g[:k], r[:k])
            only_r = np.setdiff1d(r[:k], g[:k])
            assert len(only_g) == len(only_r)
            for j in np.concatenate([only_g, only_r]):
                assert abs(s[j] - kth) <= rel * abs(kth), (b, h, int(j), float(s[j]), float(kth))
            swaps += len(only_g)
    return swaps


def decode_tolerance(ref: np.ndarray) -> float:
    """|out - ref| <= 1e-2 + 1e-2 * max|ref| (the stated decode tolerance)."""
    return 1e-2 + 1e-2 * float(np.abs(ref).max())
