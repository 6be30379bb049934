"""Two handles on two GPUs of one process.  Kernel attributes (the shared-memory size a kernel may ask for, the
L1 / shared carve-out) are per device; the launchers remember per device that they set them.  Needs two visible
GPUs; skipped otherwise."""
import numpy as np
import pytest
import torch

import paper_2302_01318_b200 as sps
import sps_synth

pytestmark = pytest.mark.gpu


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs two visible GPUs")
def test_second_device_sets_its_own_kernel_attributes():
    c = sps_synth.CONFIGS["tiny_bf16"]
    wt = sps_synth.make_weights(c["target"], tag="target")
    wd = sps_synth.make_weights(c["draft"], tag="draft")
    prompt = sps_synth.make_prompt(0, 16, c["target"]["vocab"])
    outs = []
    for dev in (0, 1):
        h = sps.Handle(c["target"], sps_synth.weights_to(wt, f"cuda:{dev}"), c["draft"], sps_synth.weights_to(wd, f"cuda:{dev}"),
                       max_seq=128, max_K=4, device=dev)
        outs.append(h.sps_generate(prompt, 32, 4, 1.0, 3)[0])
        h.close()
    assert np.array_equal(outs[0], outs[1])
