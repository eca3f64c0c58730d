"""The layer kernel's register budget, checked where it is decided: at build time (no GPU needed).

The kernel runs 352 threads per CTA with 227 KB of shared memory, one CTA per SM, and the compiler
is at the register limit that leaves (168 per thread). Two things have each cost it 4 to 15 % of its
bandwidth without failing any parity test: spills in the streaming loops, and a device function that
takes the ~1 KB parameter block by reference falling out of line, after which every thread keeps a
copy of the block on its stack and reads it from local memory. Both show in what ptxas reports."""
from paper_2609_27040_b200 import build as build_mod


def _layer_kernels():
    res = build_mod.kernel_resources()
    ks = {k: v for k, v in res.items() if "slice_layer_kernel" in k}
    assert len(ks) == 4, sorted(res)                      # tensor-core / f32 tiles x one block or several per stage
    return ks


def test_every_kernel_of_the_library_is_reported():
    res = build_mod.kernel_resources()
    for name in ("slice_layer_kernel", "copy_blocks_bulk", "copy_blocks_vector", "append_kv_kernel", "step_relay_kernel"):
        assert any(name in k for k in res), name
    for k, v in res.items():
        assert {"registers", "stack", "spill_stores", "spill_loads"} <= set(v), k


def test_layer_kernel_fits_one_cta_per_sm_without_a_stack_copy_of_its_parameters():
    for name, r in _layer_kernels().items():
        assert r["registers"] * 352 <= 65536, (name, r)  # one CTA of 352 threads per SM
        # the copy thread's bookkeeping arrays (about 200 bytes) are all the stack there is; a copy of
        # the parameter block would add about 1 KB
        assert r["stack"] <= 320, (name, r)
        assert r["spill_stores"] <= 64 and r["spill_loads"] <= 64, (name, r)


def test_the_benchmarks_variant_does_not_spill_at_all():
    # tensor-core tiles, one block per stage: 5 to 8 KV heads with grouped queries, what bench.py times
    main = [r for k, r in _layer_kernels().items() if "ILb1ELb0E" in k]
    assert len(main) == 1
    assert main[0]["spill_stores"] == 0 and main[0]["spill_loads"] == 0 and main[0]["stack"] <= 256, main[0]


def test_copy_kernels_leave_room_beside_the_layer_kernel():
    # a CTA of the 6-stage bulk gather (32 threads) shares an SM with a CTA of the layer kernel
    res = build_mod.kernel_resources()
    bulk = [r for k, r in res.items() if "copy_blocks_bulkILi6E" in k]
    layer = max(r["registers"] for r in _layer_kernels().values())
    assert len(bulk) == 1
    regs = lambda per_thread, threads: -(-per_thread * 32 // 256) * 256 * (threads // 32)   # allocated per warp, in units of 256
    assert regs(layer, 352) + regs(bulk[0]["registers"], 32) <= 65536
