"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = "".join(open(os.path.join(ROOT, "include", h)).read() for h in ("dd.h", "dd_bench.h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dd_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2607_26475_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert "dd_select_topk" in names and "dd_gather_kv_from_host" in names
    assert "dd_sparse_decode_attn" in names and "dd_decode_layer_step" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/*.h but not exported"


def test_binding_lists_the_same_entry_points_and_error_strings():
    from paper_2607_26475_b200 import build
    build.build()
    from paper_2607_26475_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    assert binding.lib.dd_strerror(0) == b"ok"
    assert binding.lib.dd_strerror(binding.DD_ERR_NOT_PINNED) == b"host memory is not page-locked"
    # size queries and configuration checks run on the host
    cfg = binding.DDConfig(32, 8, 32, 8, 128, 16, 2048, 128, 0, 2, 2, 0, 0, 0, 0, None, None, None, 0, 0, 0, None, None, 0, 0, 0)
    assert binding.lib.dd_slot_bytes(ctypes.byref(cfg)) == 64 << 20
    assert binding.lib.dd_ring_bytes(ctypes.byref(cfg)) == 128 << 20
    bad = binding.DDConfig(32, 8, 32, 8, 64, 16, 2048, 128, 0, 2, 2, 0, 0, 0, 0, None, None, None, 0, 0, 0, None, None, 0, 0, 0)
    assert binding.lib.dd_slot_bytes(ctypes.byref(bad)) == 0
    h = ctypes.c_void_p()
    assert binding.lib.dd_create(ctypes.byref(bad), ctypes.byref(h)) == binding.DD_ERR_INVALID_ARG
    assert b"head_dim" in binding.lib.dd_last_error_message(None)


def test_cluster_search_of_the_fused_selection_always_terminates():
    """The search over cluster sizes with the device queries replaced by a callback (how many clusters of a
    shape are resident at once): whatever the callback answers, the search ends; it prefers a size whose
    clusters are all resident, and returns 0 (two-kernel path) when nothing can run."""
    from paper_2607_26475_b200 import build
    build.build()
    from paper_2607_26475_b200 import binding
    ppc, smem, stages, lg = ctypes.c_int(), ctypes.c_size_t(), ctypes.c_int(), ctypes.c_int()

    def pick(max_pages, problems, rows, allow16, answer):
        calls = []

        def fits(c, sm, _):
            calls.append((c, sm))
            assert len(calls) < 32, "the search does not terminate"
            return int(answer(c, sm))
        cb = binding.PICK_FITS(fits)
        got = binding.lib.dd_test_pick_cluster(max_pages, problems, 148, rows, 4, allow16, cb, None, ctypes.byref(ppc),
                                                ctypes.byref(smem), ctypes.byref(stages), ctypes.byref(lg))
        return got, calls

    # what a B200 answers for blocks of at most 112 KiB (two per SM)
    b200 = {1: 296, 2: 148, 4: 71, 8: 33, 16: 14}
    # batch 8 x 8 KV heads, 2048 pages: 4 blocks each, 512 pages per block, logits in shared memory, 3-tile ring
    got, calls = pick(2048, 64, 1, 1, lambda c, s: b200[c])
    assert got == 4 and ppc.value == 512 and stages.value == 2 and lg.value == 0
    assert smem.value == 512 * 4 * 4 + 8 * 2 * 4096 and smem.value <= 112 * 1024
    # one request of 64K pages: 16-block clusters, logits in global scratch, every block small enough for two per SM
    got, _ = pick(65536, 8, 1, 1, lambda c, s: b200[c])
    assert got == 16 and ppc.value == 4096 and lg.value == 1 and smem.value <= 112 * 1024 and stages.value == 2
    assert pick(65536, 8, 1, 0, lambda c, s: b200[c])[0] == 8
    # 16 refused by the device: 8 is tried next, once per round
    got, calls = pick(65536, 8, 1, 1, lambda c, s: 0 if c == 16 else b200[c])
    assert got == 8 and [c for c, _ in calls][:2] == [16, 8]
    # not all clusters resident for any size: the preferred size is taken in the second round
    got, calls = pick(2048, 64, 1, 1, lambda c, s: 1)
    assert got == 4 and len(calls) <= 10
    # the case that used to loop: 128K pages with four landmarks per page, and a device that refuses everything
    got, calls = pick(131072, 8, 4, 1, lambda c, s: 0)
    assert got == 0 and len(calls) <= 10
    got, calls = pick(131072, 8, 1, 1, lambda c, s: 0)
    assert got == 0 and len(calls) <= 10
    assert pick(2048, 64, 1, 1, lambda c, s: 0)[0] == 0
    # a larger cluster is used when the preferred one cannot hold all its clusters
    got, calls = pick(2048, 64, 1, 1, lambda c, s: 64 if c >= 8 else 10)
    assert got == 8 and [c for c, _ in calls] == [4, 8]


def test_flat_work_split_of_the_tma_fed_attention_kernels():
    """Block x owns pages [x * ppb, (x + 1) * ppb) of the flat list of B * Hkv * k pages: the blocks cover the list, no
    unit is cut into more parts than reserved for it (at most 64), and large launches use every SM."""
    import ctypes
    from paper_2607_26475_b200 import binding
    rng = __import__("random").Random(3)
    shapes = [(8, 8, 128), (32, 8, 64), (8, 8, 256), (1, 8, 512), (1, 8, 16), (1, 1, 1), (1, 8, 8192), (64, 8, 3), (5, 8, 66)]
    shapes += [(rng.randint(1, 40), rng.choice([1, 2, 8]), rng.randint(1, 3000)) for _ in range(200)]
    for kind, per_sm, min_pages in ((0, 2, 8), (1, 1, 8)):
        for B, Hkv, k in shapes:
            nb, ppb, parts = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
            assert binding.lib.dd_test_attn_split(kind, B, Hkv, k, 148, ctypes.byref(nb), ctypes.byref(ppb), ctypes.byref(parts)) == 0
            nb, ppb, parts = nb.value, ppb.value, parts.value
            total = B * Hkv * k
            assert nb >= 1 and ppb >= 1 and (nb - 1) * ppb < total <= nb * ppb          # covers the list, no empty block
            assert nb <= per_sm * 148
            worst = max(((u + 1) * k - 1) // ppb - (u * k) // ppb + 1 for u in range(min(B * Hkv, 400)))
            assert worst <= parts <= 64
            ppb_free = -(-total // (per_sm * 148))                                      # without the limit on parts per unit
            if total >= per_sm * 148 * min_pages and (k - 1) // ppb_free + 2 <= 64:
                assert nb >= per_sm * 148 - per_sm * 148 // 8                          # a large launch keeps the SMs busy
    assert binding.lib.dd_test_attn_split(2, 1, 1, 1, 148, None, None, None) != 0
