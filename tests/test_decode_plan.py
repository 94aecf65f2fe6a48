"""Host logic, no GPU: the workspace that lt_workspace_bytes reports always
holds the split-KV partial slots of every launch the decode step can make.

The kernels choose the chunk length of a launch on the device, from the total
number of visible keys of that launch; the host sizes the workspace from the
shape alone.  The item count of a launch is restated here from its definition
(chunk = total keys spread over the launch's target item count, rounded up to
64 and clamped to [512, max chunk], the maximum being the larger one only for
launches of at least 2 x target x max keys; a (layer, batch row) has
ceil(n / chunk) chunks, at least one, per kv head) and swept over lengths, batch
sizes, layer ranges, masks and both pairs of maximum chunk lengths (2048 / 4096
for 16-bit caches, 8192 / 8192 for 8-bit ones); the real library's workspace size
must cover it every time.  The same sweep checks the per-layer bound behind
lt_decode_step_layers: a launch over k layers never has more than k times the
slots that the layered workspace keeps for every layer.
"""
import numpy as np
import pytest

import paper_2410_13846_b200 as lt

HEADER, ALIGN = 256, 256
MIN_CHUNK, TARGET_ITEMS, MAX_ENTRIES = 512, 592, 2048


def _round_up(x, a):
    return (x + a - 1) // a * a


def items_of_launch(n_visible, hkv, grid, max_chunk, mid_chunk):
    """Items (= partial slots) of one launch over (layer, batch row) pairs with the
    given visible lengths, as the kernels derive them.  `hkv` counts the units of a
    (layer, batch row): its kv heads."""
    total_keys = sum(n_visible) * hkv
    target = min(grid * 8, TARGET_ITEMS)
    c = -(-total_keys // target) if total_keys else 0
    c = _round_up(c, 64)
    hi = max_chunk if total_keys >= 2 * TARGET_ITEMS * max_chunk else mid_chunk   # the longest chunks only for large launches
    chunk = max(MIN_CHUNK, min(hi, c))
    return sum(hkv * max(1, -(-n // chunk)) for n in n_visible), chunk


def slots_in_workspace(shape):
    """Partial slots that the workspace reported by the library has room for."""
    G = shape.n_q_heads // shape.n_kv_heads
    nbytes = lt.workspace_bytes(shape, 0, 0)
    units = shape.n_layers * shape.batch * shape.n_kv_heads
    prefix = HEADER + _round_up((units + 2 * shape.n_layers) * 4, ALIGN)   # unit counters + a counter pair per layer
    per_slot = G * 2 * 4 + G * shape.head_dim * 4      # a slot holds (max, sum) and O of every head of the group
    # two regions of 4-byte words, each rounded up to the alignment (at most ALIGN - 4 bytes of padding each):
    # slots * per_slot >= bytes - prefix - 2 * (ALIGN - 4)
    return -(-(nbytes - prefix - 2 * (ALIGN - 4)) // per_slot), (nbytes - prefix) // per_slot


@pytest.mark.parametrize("fp8", [0, 1])
def test_workspace_covers_every_launch(fp8):
    g = np.random.default_rng(5 + fp8)
    max_chunk, mid_chunk = (8192, 8192) if fp8 else (4096, 2048)
    worst = 0.0
    for trial in range(400):
        L = int(g.choice([1, 2, 3, 8, 32, 64, 128]))
        B = int(g.choice([1, 2, 3, 8, 32, 100]))
        Hkv = int(g.choice([1, 2, 8]))
        G = int(g.choice([1, 4, 5, 8] if fp8 else [1, 4, 5, 8, 12, 16]))
        S = int(g.choice([0, 4, 64]))
        R = int(g.choice([1, 60, 2044, 4092, 20000]))
        cap = int(g.choice([1, 17, 511, 512, 513, 2047, 2048, 2049, 4097, 32768 + 128, 70000, 131072 + 4]))
        shape = lt.Shape(L, B, Hkv * G, Hkv, 128, S, R, cap, lt.LT_BF16, kv_fp8=fp8,
                         kv_scales=None)
        if fp8:
            # the size query only validates that a scale table is given; any non-null address will do on the host
            class _Fake:
                is_cuda, dtype = True, __import__("torch").float32
                def is_contiguous(self): return True
                def data_ptr(self): return 0x1000
            shape.kv_scales = _Fake()
        lo_slots, _ = slots_in_workspace(shape)
        # lt_decode_step_layers gives every layer its own slots: most items per layer of any launch
        n_max = max(cap, S + R)
        per_layer = max(TARGET_ITEMS + B * Hkv, B * Hkv * -(-n_max // mid_chunk))
        units = L * B * Hkv
        layered_need = (HEADER + _round_up((units + 2 * L) * 4, ALIGN) + _round_up(per_layer * L * G * 2 * 4, ALIGN)
                        + _round_up(per_layer * L * G * 128 * 4, ALIGN))
        assert lt.workspace_bytes_layers(shape, 0, 0) >= max(layered_need, lt.workspace_bytes(shape, 0, 0))
        C = S + R
        layers_per_launch = max(1, MAX_ENTRIES // B)
        for _ in range(6):
            kind = g.integers(4)
            mask = (g.random(L) < [0.0, 1.0, 0.5, 0.25][kind]).astype(int)
            len_kind = g.integers(4)
            if len_kind == 0:
                lens = np.full(B, cap)                                     # every row full
            elif len_kind == 1:
                lens = g.integers(0, cap + 1, size=B)                      # ragged
            elif len_kind == 2:
                lens = np.full(B, min(cap, int(g.choice([0, 1, 511, 512, 513, 2048, 2049]))))
            else:
                lens = np.minimum(cap, g.integers(0, 3, size=B) * max_chunk + g.integers(-1, 2, size=B)).clip(0)
            begin = int(g.integers(0, L))
            count = int(g.integers(1, L - begin + 1))
            for grid in (148, 296, 1, 37):
                for done in range(0, count, layers_per_launch):
                    layers = range(begin + done, begin + min(count, done + layers_per_launch))
                    n_vis = [min(int(n), C if mask[l] else cap) for l in layers for n in lens]
                    items, chunk = items_of_launch(n_vis, Hkv, grid, max_chunk, mid_chunk)
                    assert items <= lo_slots, (trial, L, B, Hkv, G, cap, C, chunk, items, lo_slots)
                    assert items <= per_layer * len(layers), (trial, L, B, Hkv, cap, C, chunk, items, per_layer)
                    worst = max(worst, items / max(lo_slots, 1))
    assert worst > 0.5          # the sweep does get near the bound: the bound is not vacuous


def test_restated_item_count_on_the_benchmark_stack():
    """The 32K benchmark stack: 16 full layers x 8 rows x 8 kv heads x 9 chunks of
    <= 4096 keys + 16 lazy layers with one chunk per (row, kv head); one of its layers alone: 2048-key chunks."""
    n = 32768 + 64
    n_vis = [n] * (16 * 8) + [2048] * (16 * 8)
    items, chunk = items_of_launch(n_vis, 8, 296, 4096, 2048)
    assert chunk == 4096 and items == 16 * 8 * 8 * 9 + 16 * 8 * 8
    items, chunk = items_of_launch([n] * 8, 8, 296, 4096, 2048)
    assert chunk == 2048 and items == 8 * 8 * 17
    # a one-layer call over 3000 keys picks the shortest chunks
    items, chunk = items_of_launch([3000], 2, 296, 4096, 2048)
    assert chunk == 512 and items == 2 * 6
