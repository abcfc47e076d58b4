"""HostPipeline without a device: it must refuse loudly (there is no CPU path), and bad arguments are rejected first."""
import pytest
import torch

from paper_2303_08999_b200.hostpipe import HostPipeline


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the behaviour on a machine without a GPU")
def test_needs_a_device():
    with pytest.raises(RuntimeError, match="CUDA"):
        HostPipeline({"lr": ((1, 3, 4, 4), torch.float32)}, {"out": ((1, 3, 16, 16), torch.float32)})
