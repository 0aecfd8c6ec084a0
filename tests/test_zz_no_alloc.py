"""The allocation-free rescale (fesc_rescale_static) against fesc_rescale.

Some callers of the library cannot allocate device memory inside a call: they run under a memory budget
owned by another allocator, in a loop that cannot take an allocation's device-wide synchronisation, or inside
a host that forbids allocator calls.  For them the library offers a rescale whose scratch is a fixed array in the library image.
This file checks, through the C ABI, that it returns exactly what fesc_rescale returns (integer residues, so
bit for bit), twice in a row on different data (the array is shared and keeps the previous call's contents),
that it equals the CPU oracle's rescale, that a call made after the context's own scratch arena has been given
back leaves both the arena and the device's free memory untouched (the property the entry point exists for),
and that a batch beyond the array's size is refused with a clear error.  It is collected last on purpose.
"""
import numpy as np
import pytest

from tests.gpu_util import ctx_pair, random_ct, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,level,batch", [("small", 24, 5), ("full", 24, 3)])
def test_static_rescale_matches_rescale_twice(name, level, batch):
    import torch

    ctx, orc, _ = ctx_pair(name)
    for call in range(2):
        ct = to_dev(random_ct(orc, 90 + call, level, level, batch))
        want = torch.empty((batch, 2, level - 1, orc.N), dtype=torch.int64, device="cuda")
        got = torch.full_like(want, -1)
        ctx.rescale(ct, want, batch, level)
        ctx.rescale_static(ct, got, batch, level)
        ctx.sync()
        assert torch.equal(got, want), (name, call)
    # a lower level right after, so stale rows of the larger call are still in the array
    ct = to_dev(random_ct(orc, 95, 3, 3, 1))
    want = torch.empty((1, 2, 2, orc.N), dtype=torch.int64, device="cuda")
    got = torch.full_like(want, -1)
    ctx.rescale(ct, want, 1, 3)
    ctx.rescale_static(ct, got, 1, 3)
    ctx.sync()
    assert torch.equal(got, want)


def test_static_rescale_matches_the_oracle_and_allocates_nothing():
    """After a warm-up call (the first call on a device looks up the array and loads its module) the context's
    arena is returned to the driver; a further call must then leave the arena at zero bytes and the free device
    memory unchanged, and its result must equal the oracle's rounded division by the last prime."""
    import torch

    ctx, orc, _ = ctx_pair("small")
    level, batch = 7, 3
    cts = random_ct(orc, 97, level, level, batch)
    ct = to_dev(cts)
    got = torch.full((batch, 2, level - 1, orc.N), -1, dtype=torch.int64, device="cuda")
    ctx.rescale_static(ct, got, batch, level)          # warm-up: symbol lookup, module load
    ctx.sync()
    ctx.trim()
    assert ctx.counters()[3] == 0
    got.fill_(-1)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ctx.rescale_static(ct, got, batch, level)
    ctx.sync()
    assert ctx.counters()[3] == 0                       # the arena was not grown
    assert torch.cuda.mem_get_info()[0] == free_before  # and nothing else was taken from the device
    want = np.stack([orc.rescale(c) for c in cts])
    assert np.array_equal(got.cpu().numpy().view(np.uint64), want)


def test_static_rescale_rejects_oversized_batch():
    import torch
    import paper_2608_17442_b200 as fesc

    ctx, orc, _ = ctx_pair("full")
    ct = torch.zeros((5, 2, 2, orc.N), dtype=torch.int64, device="cuda")   # 5 * 2 * 65536 words > 524288
    out = torch.zeros((5, 2, 1, orc.N), dtype=torch.int64, device="cuda")
    with pytest.raises(fesc.FescError) as e:
        ctx.rescale_static(ct, out, 5, 2)
    assert e.value.code == fesc.EINVAL and "static scratch" in str(e.value)
