"""The allocation-free greedy-acceptance entry point against the regular one.

Some callers cannot give the library a workspace (their framework owns all device memory, or they
are only lent input and output tensors), so beagle_verify_greedy_static keeps its scratch in a
device array built into the library.  Its answers must be those of beagle_verify_greedy, on
back-to-back calls too: the second call finds the first call's leftovers in the shared array.
This file sorts last so that an earlier failure never hides behind it.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2505_24544_b200 import workloads as WL


def test_oversize_request_is_rejected_with_a_message_on_the_host():
    from paper_2505_24544_b200 import build
    from paper_2505_24544_b200.binding import load_library
    build.build()
    lib = load_library()
    err = C.create_string_buffer(256)
    # 65 * 64 = 4160 rows fit exactly; one more sequence does not.  Rejected before any CUDA call.
    assert lib.beagle_verify_greedy_static(66, 63, 1000, None, None, 0, None, None, None, err, len(err)) == 3
    assert b"4224" in err.value and b"4160" in err.value
    assert lib.beagle_verify_greedy_static(1, 1, 0, None, None, 0, None, None, None, err, len(err)) == 1
    assert lib.beagle_verify_greedy_static(0, 4, 1000, None, None, 0, None, None, None, None, 0) == 0


@pytest.mark.gpu
def test_static_scratch_variant_matches_regular_entry_point_twice():
    from paper_2505_24544_b200.binding import BeagleHead, beagle_verify_greedy_static
    w = WL.WORKLOADS["c1_tiny_fp32"]
    head = BeagleHead.from_workload(w, WL.make_weights(w))
    rng = WL.data_rng(w, 1234)
    # two calls in a row with different shapes and dtypes: the second reuses the array's stale contents
    for batch, gamma, dt in ((7, 5, "fp32"), (3, 8, "bf16")):
        draft = WL.make_tokens(w, rng, (batch, gamma))
        planted = np.concatenate([draft, np.full((batch, 1), -1)], axis=1)
        for b in range(batch):
            planted[b, rng.integers(0, gamma + 1):] = -1        # agree on a random-length prefix
        logits = WL.make_target_logits(w, rng, batch * (gamma + 1), planted.reshape(-1))
        logits = WL.round_to_storage(logits.reshape(-1), dt).reshape(batch, gamma + 1, w.vocab)
        lg = torch.from_numpy(logits).cuda().to(torch.bfloat16 if dt == "bf16" else torch.float32)
        d = torch.from_numpy(draft).cuda()
        acc_ref, out_ref = head.verify_greedy(d, target_logits=lg)
        acc = torch.full((batch,), -7, dtype=torch.int32, device="cuda")
        out = torch.full((batch, gamma + 1), -7, dtype=torch.int32, device="cuda")
        beagle_verify_greedy_static(d, lg, acc, out)
        torch.cuda.synchronize()
        assert torch.equal(acc, acc_ref) and torch.equal(out, out_ref)      # integer results: bit-exact
        assert int(acc.max()) > 0
