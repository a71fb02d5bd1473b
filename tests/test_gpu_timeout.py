"""The give-up path of the device-side waits: every wait in the library is bounded; this makes one run out."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_13915_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """A wait that nothing satisfies runs out of its (short) budget, the status word says MSD_ERR_TIMEOUT, the kernel has
    ended by itself, and the library keeps working afterwards."""
    stream = torch.cuda.current_stream().cuda_stream
    assert binding.lib().msd_debug_timeout_selftest(2_000_000, stream) == 0       # about a millisecond of SM clocks
    torch.cuda.synchronize()
    with pytest.raises(binding.MsdError) as err:
        binding.last_device_status()
    assert "TIMEOUT" in str(err.value)
    binding.last_device_status()                                                   # the word was cleared by the read
    c = inputs.gemm_w8_case(8, 256, 512, seed=3)
    x = torch.from_numpy(np.ascontiguousarray(c.x).view(np.int16)).view(torch.bfloat16).cuda()
    y, acc = binding.gemm_w8a16(x, torch.from_numpy(c.w).cuda(), torch.from_numpy(c.w_scale).cuda(), out_dtype=torch.float32,
                                want_acc=True)
    torch.cuda.synchronize()
    binding.last_device_status()
    _, oacc = oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64", want_acc=True)
    assert np.array_equal(acc.cpu().numpy(), oacc)
