"""The allocation-free entry point against the ordinary handle-based path.

mava_rollout_run_static serves callers that may not allocate device memory while they run (all
memory already in their own pool, or a loop that cannot afford the device-wide synchronisation of
cudaMalloc/cudaFree): its scratch is a static device array inside the library.  The test calls it
twice in a row through the C ABI -- the array keeps the first call's contents, so the second call
shows that stale scratch does no harm -- and compares every output with what create + run write
for a fresh handle.  It is collected last on purpose.
"""
import ctypes as C

import numpy as np
import pytest

from paper_2107_01460_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx,precision,n_envs,T", [(1, binding.MAVA_PRECISION_BF16, 300, 40),
                                                    (4, binding.MAVA_PRECISION_BF16, 70, 20),
                                                    (3, binding.MAVA_PRECISION_FP32, 50, 20)])
def test_static_scratch_rollout_matches_handle_rollout(idx, precision, n_envs, T):
    import torch

    w = wl.workload(idx)
    cfg = binding.make_config(w, precision=precision, flags=binding.MAVA_FLAG_WRITE_LOGITS, max_T=T, n_envs=n_envs)
    params = torch.from_numpy(wl.make_params(w, bias_scale=0.1)).cuda()
    ref = binding.Rollout(cfg)
    ref.run(params, T)
    assert ref.status() == binding.MAVA_OK
    names = ("obs", "actions", "logp", "values", "rewards", "dones", "logits")
    want = {n: getattr(ref, n).clone() for n in names}

    # caller-owned outputs, allocated before the calls under test
    out = {n: torch.full_like(want[n], 7) for n in names}
    bufs = binding.mava_buffers_t(out["obs"].data_ptr(), out["actions"].data_ptr(), out["logp"].data_ptr(),
                                  out["values"].data_ptr(), out["rewards"].data_ptr(), out["dones"].data_ptr(),
                                  None, None, out["logits"].data_ptr())
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):
        for t in out.values():
            t.fill_(7)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = binding.mava_rollout_run_static(cfg, bufs, params.data_ptr(), T, stream)
        free_after = torch.cuda.mem_get_info()[0]
        assert rc == binding.MAVA_OK, binding.strerror(rc)
        # the same kernels on the same inputs: the same bits in every array
        for n in names:
            assert torch.equal(out[n], want[n]), (call, n)
        # the first call on a device may make the driver load the module that holds the array; from then on the
        # device's free memory must not move across a call
        if call == 1:
            assert free_after >= free_before, (free_before, free_after)


def test_static_scratch_rejects_what_does_not_fit():
    w = wl.workload(4)
    cfg = binding.make_config(w, precision=binding.MAVA_PRECISION_BF16)  # 32768 envs: beyond the array
    bufs = binding.mava_buffers_t(*([256] * 9))  # never dereferenced: the size check comes first
    assert binding.mava_rollout_run_static(cfg, bufs, 256, 1, None) == binding.MAVA_ERR_CAPACITY
    small = binding.make_config(w, precision=binding.MAVA_PRECISION_BF16, n_envs=64, max_T=4)
    assert binding.mava_rollout_run_static(small, bufs, 256, 5, None) == binding.MAVA_ERR_CAPACITY
    assert binding.mava_rollout_run_static(small, bufs, 0, 1, None) == binding.MAVA_ERR_INVALID_ARG
