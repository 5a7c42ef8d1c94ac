"""scout_sign_chunks_noalloc against the CPU oracle and against scout_sign_chunks.

The no-allocation entry point is for callers that cannot allocate device memory
at the moment they need a check: code running inside a training step whose
framework already owns nearly all of HBM, or a handler that runs after an
out-of-memory error.  It must produce the records of the planned entry point
for a one-tensor-per-replica state: hashes and counts identical to the oracle's
and to the planned entry point's, fp64 sums within the tolerance the other parity
tests use.  Two calls in a row share the library's fixed scratch array, so the
second call runs on different data and must not see anything of the first.
This file sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

import helpers
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def _host(views):
    return [[v.cpu() for v in rep] for rep in views]


def _oracle(w, views):
    """Oracle records plus sum|x| per (chunk, replica), the scale of the tolerance on the sums."""
    hv = _host(views)
    sigs, chunks = helpers.oracle_sign_all(w, hv)
    return sigs, helpers.chunk_abs_sums(w, hv, chunks)


def _planned(w, views):
    """Records of the planned entry point."""
    plan = helpers.gpu_plan(w)
    plan.bind(views)
    plan.sign()
    torch.cuda.synchronize()
    from paper_2608_11034_b200 import binding
    sigs = plan.d_sigs.cpu().numpy().view(binding.SIG_DTYPE).reshape(plan.C, w.R).copy()
    plan.close()
    return sigs


def _noalloc(w, views):
    from paper_2608_11034_b200 import binding
    s = w.specs[0]
    C = (s.nbytes + w.chunk_bytes - 1) // w.chunk_bytes
    # the records are followed by a guard band nothing may write to
    d_sigs = torch.full((C * w.R * 32 + 256,), 0xAB, dtype=torch.uint8, device="cuda")
    binding.scout_sign_chunks_noalloc(w.R, [views[r][0].data_ptr() for r in range(w.R)], s.nbytes,
                                      binding.DTYPE_CODE[s.dtype], helpers.shape_tags(w)[0],
                                      w.chunk_bytes, d_sigs.data_ptr(),
                                      torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    host = d_sigs.cpu().numpy()
    assert (host[C * w.R * 32:] == 0xAB).all(), "write past the end of the record table"
    assert binding.scout_noalloc_guards_ok(), "write outside the fixed scratch array"
    return host[:C * w.R * 32].view(binding.SIG_DTYPE).reshape(C, w.R)


def test_two_calls_in_a_row_match_the_oracle_and_the_planned_entry_point():
    # first call: fp32, ragged tail, one NaN and one flipped bit
    w1 = inputs.Workload("noalloc_f32", 0, "x", 3, 64 << 10,
                         [inputs.TensorSpec("x", (1_000_003,), "f32", "normal", 0.02)], 41)
    _, v1 = inputs.generate(w1, "cuda")
    inputs.apply_patches(v1, w1.specs, [inputs.Patch(1, 0, 77_777, "xor", 1 << 9),
                                        inputs.Patch(2, 0, 999_999, "set", 0x7FC00000)])
    got1 = _noalloc(w1, v1)
    # second call right after it: other dtype, other size, other chunking, more replicas
    w2 = inputs.Workload("noalloc_bf16", 0, "x", 5, 1 << 20,
                         [inputs.TensorSpec("g", (3_333_337,), "bf16", "normal", 1e-3)], 42)
    _, v2 = inputs.generate(w2, "cuda")
    inputs.apply_patches(v2, w2.specs, [inputs.Patch(4, 0, 3_000_000, "xor", 1 << 3)])
    got2 = _noalloc(w2, v2)
    # and the first input once more: the shared scratch keeps nothing that matters
    got1_again = _noalloc(w1, v1)

    o1, abs1 = _oracle(w1, v1)
    o2, abs2 = _oracle(w2, v2)
    helpers.assert_sigs_match(got1, o1, abs1)
    helpers.assert_sigs_match(got2, o2, abs2)
    helpers.assert_sigs_match(got1, _planned(w1, v1), abs1)
    helpers.assert_sigs_match(got2, _planned(w2, v2), abs2)
    assert got1.tobytes() == got1_again.tobytes()
    assert int(got1["nan_count"].sum()) == 1
    assert (got1["hash"][:, 0] != got1["hash"][:, 1]).sum() == 1
    assert (got2["hash"][:, 0] != got2["hash"][:, 4]).sum() == 1


@pytest.mark.parametrize("name,dtype,numel,chunk_bytes,R", [
    # 256 MB per replica: the 2, 4 and 8 KiB tiles need more records than the fixed array
    # holds, so the entry point escalates to 16 KiB tiles; 66,048-byte chunks are not a
    # multiple of that tile (4 full tiles and a 512-byte one per chunk)
    ("big_odd_chunks", "f32", 64_000_037, 66_048, 3),
    # the same size with 4 MiB chunks: 256 tiles per chunk through the strided combine
    ("big_even_chunks", "bf16", 128_000_001, 4 << 20, 3),
    # chunks smaller than the smallest tile: one short tile per chunk
    ("tiny_chunks", "f32", 300_001, 512, 4),
    ("tiny_chunks_i64", "i64", 50_001, 1536, 2),
])
def test_tile_escalation_and_chunk_shapes_against_the_oracle(name, dtype, numel, chunk_bytes, R):
    dist = "randint40" if dtype == "i64" else "normal"
    w = inputs.Workload("noalloc_" + name, 0, "x", R, chunk_bytes,
                        [inputs.TensorSpec("x", (numel,), dtype, dist, 0.02)], 43)
    _, v = inputs.generate(w, "cuda")
    es = inputs.DTYPE_BYTES[dtype]
    last_chunk_first_elem = (w.specs[0].nbytes // chunk_bytes) * chunk_bytes // es
    patches = [inputs.Patch(R - 1, 0, numel // 3, "xor", 1 << 5),
               inputs.Patch(0, 0, min(numel - 1, last_chunk_first_elem), "xor", 1)]
    if dtype in ("f32", "bf16"):
        patches.append(inputs.Patch(1, 0, numel - 1, "set", 0x7F800000 if dtype == "f32" else 0x7F80))
    inputs.apply_patches(v, w.specs, patches)
    got = _noalloc(w, v)
    want, abs_sums = _oracle(w, v)
    helpers.assert_sigs_match(got, want, abs_sums)
    if dtype in ("f32", "bf16"):
        assert int(got["inf_count"].sum()) == 1 and int(got["inf_count"][-1, 1]) == 1
    # a call that is not the first on this device takes no device memory: the driver's
    # free-memory figure is the same before and after it (torch's own buffers were all
    # allocated before the first reading and are still held)
    d_sigs = torch.empty(got.size * 32, dtype=torch.uint8, device="cuda")
    from paper_2608_11034_b200 import binding
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    binding.scout_sign_chunks_noalloc(R, [v[r][0].data_ptr() for r in range(R)], w.specs[0].nbytes,
                                      binding.DTYPE_CODE[dtype], helpers.shape_tags(w)[0], chunk_bytes,
                                      d_sigs.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    free2, _ = torch.cuda.mem_get_info()
    assert free2 == free1, (free1, free2)


def test_sizes_beyond_the_fixed_scratch_are_rejected_without_launching():
    from paper_2608_11034_b200 import binding
    x = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    d_sigs = torch.zeros(64, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    with pytest.raises(binding.ScoutError) as e:      # 64 replicas x 8 GiB: far over the limit
        binding.scout_sign_chunks_noalloc(64, [x.data_ptr()] * 64, 8 << 30, binding.DT_U8, 0,
                                          1 << 30, d_sigs.data_ptr(), s)
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.ScoutError) as e:
        binding.scout_sign_chunks_noalloc(3, [x.data_ptr() + 8] * 3, 1024, binding.DT_U8, 0, 512,
                                          d_sigs.data_ptr(), s)
    assert e.value.code == binding.ERR_ALIGN
    torch.cuda.synchronize()
