"""The GEMM entry point that allocates nothing: split-K scratch in the library's fixed device array.

Collected last on purpose. It serves callers that have no arena to hand over and may not call the
allocator (a serving loop that must not stall, a plugin under a host framework's memory accounting, a
process with a budget fixed at start-up). The checks: its output agrees with the fp64 oracle and with the
planned path (fluid_plan + fluid_run on a one-LINEAR graph) within the tolerance the other GEMM tests use,
on two calls in a row that share the static array, the second smaller than the first; free device memory
does not move; the status word reads clean after each call."""
import numpy as np
import pytest

from paper_2411_09242_b200 import fluid, synth
from tests.helpers import assert_close, ensure_lib, rand_feed, run_gpu, run_oracle, single_op_graph


def test_bad_arguments_are_refused_before_any_device_work():
    """Both refusals below are decided from the arguments alone (no device query, no launch), so made-up
    addresses never reach a kernel."""
    ensure_lib()
    with pytest.raises(fluid.FluidError) as e:          # K not a multiple of 8
        fluid.fluid_gemm_bf16_static_scratch(0x1000, 0x2000, 0, 0x3000, 128, 768, 100)
    assert e.value.code == fluid.FLUID_EINVAL
    with pytest.raises(fluid.FluidError) as e:          # misaligned operand
        fluid.fluid_gemm_bf16_static_scratch(0x1008, 0x2000, 0, 0x3000, 128, 768, 1024)
    assert e.value.code == fluid.FLUID_EALIGN


@pytest.mark.gpu
def test_sizes_beyond_the_static_array_are_rejected():
    """How far a shape is split depends on the SM count of the device, so this runs on the device with real
    buffers: were the shape accepted, the launch would be a legal one."""
    import torch
    ensure_lib()
    M, N, K = 128, 2432, 4096   # 148 SMs: 19 tiles of 128x128, split 7 ways, 64 KiB each = 8.7 MB > 8 MiB
    a = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    b = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
    c = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    if torch.cuda.get_device_properties(0).multi_processor_count < 140:
        pytest.skip("the shape is sized for the split a 148-SM device chooses")
    with pytest.raises(fluid.FluidError) as e:
        fluid.fluid_gemm_bf16_static_scratch(a.data_ptr(), b.data_ptr(), 0, c.data_ptr(), M, N, K,
                                             torch.cuda.current_stream().cuda_stream)
    assert e.value.code == fluid.FLUID_EINVAL and "static array holds" in str(e.value)
    torch.cuda.synchronize()


@pytest.mark.gpu
def test_two_calls_in_a_row_match_the_oracle_and_the_planned_path():
    import torch
    ensure_lib()
    free_before = None
    for call, (M, N, K, with_bias) in enumerate([(128, 768, 3072, True), (96, 256, 2048, False)]):
        shapes = [[M, K], [K, N]] + ([[N]] if with_bias else [])
        g = single_op_graph(synth.LINEAR, shapes, [M, N], synth.BF16, {"contract": 1},
                            in_kinds={1: synth.CONST, 2: synth.CONST})
        feeds = {0: rand_feed([M, K], synth.BF16, 31 + call), 1: rand_feed([K, N], synth.BF16, 41 + call)}
        if with_bias:
            feeds[2] = rand_feed([N], synth.BF16, 51)
        want = run_oracle(g, feeds)[g.outputs[0]]                                   # the plain definition, fp64
        planned, plan, _ = run_gpu(g, feeds, synth.default_candidates(g))          # the existing entry points
        a = fluid.to_device(feeds[0], synth.BF16)
        b = fluid.to_device(np.ascontiguousarray(feeds[1].T), synth.BF16)            # [N, K], k contiguous
        bias = fluid.to_device(feeds[2], synth.BF16) if with_bias else None
        c = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        torch.cuda.synchronize()
        if call == 1:
            free_before = torch.cuda.mem_get_info()[0]
        stream = torch.cuda.current_stream().cuda_stream
        fluid.fluid_gemm_bf16_static_scratch(a.data_ptr(), b.data_ptr(), bias.data_ptr() if with_bias else 0,
                                             c.data_ptr(), M, N, K, stream)
        assert fluid.fluid_static_scratch_status(stream) == 0                        # synchronises; no wait gave up
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before                       # nothing was allocated
        got = c.float().cpu().numpy().astype(np.float64)
        assert_close(got, want, synth.BF16, f"static-scratch GEMM call {call} vs oracle", tol=2 ** -7)
        assert_close(got, planned[g.outputs[0]], synth.BF16, f"static-scratch GEMM call {call} vs planned path",
                     tol=2 ** -7)
        plan.close()
