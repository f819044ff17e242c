"""Test-only helpers: pack dense per-trajectory K/V into a paged pool, bf16 bit conversions."""
import numpy as np
import torch


def to_bf16_bits(x) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    w = b.astype(np.uint32) << 16
    return w.view(np.float32).astype(np.float64)


def pack_pages(K_list, V_list, P, num_kv_heads, D, rng=None, spare=3, fill_bits=0x7FC0, table_fill=-1,
               max_pages=None):
    """K_list[t], V_list[t]: uint16 [L_t][Hkv][D].  Returns (k_pool, v_pool, table, lens).
    Physical pages are a random permutation when rng is given, else in order; all slots not
    written hold fill_bits (NaN by default)."""
    T = len(K_list)
    lens = np.array([k.shape[0] for k in K_list], dtype=np.int32)
    pages = (lens + P - 1) // P
    total = int(pages.sum())
    num_pages = total + spare
    ids = rng.permutation(num_pages)[:total] if rng is not None else np.arange(total)
    mp = max(1, int(pages.max()) if T else 1) if max_pages is None else max_pages
    table = np.full((T, mp), table_fill, dtype=np.int32)
    k_pool = np.full((num_pages, num_kv_heads, P, D), fill_bits, dtype=np.uint16)
    v_pool = np.full((num_pages, num_kv_heads, P, D), fill_bits, dtype=np.uint16)
    o = 0
    for t in range(T):
        table[t, :pages[t]] = ids[o:o + pages[t]]
        o += int(pages[t])
        for j in range(int(lens[t])):
            pg = table[t, j // P]
            k_pool[pg, :, j % P, :] = K_list[t][j]
            v_pool[pg, :, j % P, :] = V_list[t][j]
    return k_pool, v_pool, table, lens
