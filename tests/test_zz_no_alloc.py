"""The allocation-free decode entry point against the regular one.

idxc_indexer_decode_noalloc serves hosts that cannot give the library a workspace (all HBM
already owned by a KV-cache pool, or no allocation allowed inside the decode loop): its score
scratch is an array inside the library. It runs the same kernels as idxc_indexer_decode, so the
indices must be identical. Two calls in a row with different sequence lengths check that
whatever the first call left in the shared array does not leak into the second. Collected last
so that a failure here cannot hide any other test.
"""
import pytest
import torch

from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _regular(x, k_top):
    B, H, d = x.q_step.shape
    out = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, x.max_len, H, d, k_top), DEV)
    idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, x.q_scale, x.k_scale,
                        topk_out=out, workspace=ws)
    return out


def _noalloc(x, k_top):
    B = x.q_step.shape[0]
    out = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_decode_noalloc(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, out,
                                x.q_scale, x.k_scale)
    return out


def _case(seed, lens, fp8=False):
    x = synth.decode_inputs(len(lens), 64, 128, 0, 0, seed=seed, fp8=fp8, lens=lens)
    for name in ("q_step", "k_cache", "w", "q_scale", "k_scale", "k_offsets", "lens"):
        v = getattr(x, name)
        if v is not None:
            setattr(x, name, v.to(DEV))
    return x


def test_noalloc_decode_matches_regular_entry_point_twice_in_a_row():
    k_top = 256
    first = _case(41, [9000, 300, 4097, 12345])          # long rows fill the shared array
    second = _case(42, [700, 5000, 129])                 # shorter rows land on top of the old scores
    got1 = _noalloc(first, k_top)
    got2 = _noalloc(second, k_top)
    idxc.poll_device_status()
    assert torch.equal(got1, _regular(first, k_top))
    assert torch.equal(got2, _regular(second, k_top))
    third = _case(43, [2500, 64], fp8=True)
    assert torch.equal(_noalloc(third, 128), _regular(third, 128))


def test_noalloc_decode_allocates_nothing_after_its_first_call_on_a_device():
    """The first call on a device makes the driver create the built-in array and load the decode kernels; from then on
    a call must leave the device's free memory untouched, whatever head count, dtype or batch shape it brings (a
    serving host makes the first call at start-up, then hands the rest of HBM to its cache pool). Outputs and inputs
    are allocated before the free memory is read, so only the library's own behaviour is measured."""
    warm = _case(51, [300, 40])
    out_w = torch.full((2, 8), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_decode_noalloc(warm.q_step, warm.k_cache, warm.w, warm.k_offsets, warm.lens, warm.max_len, 8, out_w,
                                warm.q_scale, warm.k_scale)                      # first call (unless an earlier test made it)
    idxc.poll_device_status()
    cases = []
    for seed, (H, d, fp8, lens, k_top) in enumerate([(16, 64, False, [5000, 129], 32), (32, 128, True, [700], 64),
                                                       (64, 128, False, [20000, 17000, 300], 2048), (64, 64, False, [9, 2000], 16)]):
        x = synth.decode_inputs(len(lens), H, d, 0, 0, seed=60 + seed, fp8=fp8, lens=lens)
        for name in ("q_step", "k_cache", "w", "q_scale", "k_scale", "k_offsets", "lens"):
            v = getattr(x, name)
            if v is not None:
                setattr(x, name, v.to(DEV))
        cases.append((x, k_top, torch.full((len(lens), k_top), -7, dtype=torch.int32, device=DEV)))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for x, k_top, out in cases:
        idxc.indexer_decode_noalloc(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, out, x.q_scale, x.k_scale)
    idxc.poll_device_status()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, f"free device memory moved by {free_before - free_after} bytes"
    for x, k_top, out in cases:
        assert torch.equal(out, _regular(x, k_top))


def test_noalloc_decode_rejects_steps_larger_than_its_array():
    x = _case(44, [100, 200])
    out = torch.empty((2, 16), dtype=torch.int32, device=DEV)
    too_long = idxc.NOALLOC_SCRATCH_BYTES // (2 * 4) + 32          # 2 rows of that many floats no longer fit
    with pytest.raises(idxc.IdxcError) as e:
        idxc.indexer_decode_noalloc(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, too_long, 16, out)
    assert e.value.status == idxc.ERR_WORKSPACE
    # the largest step that fits is accepted (lens stay small; only the bound is large)
    fits = idxc.NOALLOC_SCRATCH_BYTES // (2 * 4)
    idxc.indexer_decode_noalloc(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, fits, 16, out)
    idxc.poll_device_status()
    assert torch.equal(out, _regular(x, 16))
