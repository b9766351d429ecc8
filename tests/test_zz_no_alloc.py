"""The allocation-free routing entry point against the regular step.

Some hosts hand all device memory to their own arena, or cannot afford the device-wide
synchronisation of cudaMalloc inside the decode loop; for them the library offers
``oled_route_noalloc``, whose scratch is a fixed array inside the library.  This test calls it
through the C ABI twice in a row, with different inputs (so stale contents of the shared array
would show), and checks every output bit for bit against what ``oled_denoise_step`` produced
for the same inputs and against the CPU oracle's gate, top-k and permutation of the same bits.  It is collected last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import moe_layer as oracle_moe  # noqa: E402
from paper_2609_33385_b200 import synth  # noqa: E402

pytestmark = pytest.mark.gpu


def test_route_noalloc_matches_denoise_step_twice_in_a_row():
    from paper_2609_33385_b200 import binding, build
    build.build()
    from paper_2609_33385_b200.runner import StackRunner, bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=8, top_k=3, hidden=512)
    run = StackRunner(w, capacity=[4], max_tokens=64)
    dev = run.device
    e, k, h = w.n_experts, w.top_k, w.hidden
    wr_dev, _ = run._router_dev[0]
    stream = torch.cuda.current_stream(dev).cuda_stream
    try:
        for call, n in enumerate((37, 9)):                # second call is smaller: stale rows would show
            h_bits, conf = synth.flat_tokens(w, n, 40 + call)
            x, c = bits_to_dev(h_bits, dev), torch.from_numpy(conf).to(dev)
            out = torch.empty((n, h), dtype=torch.bfloat16, device=dev)
            run.step(0, x, c, out)
            ref = run.ctx.debug_last(0, n)

            ids = torch.full((n * k,), -1, dtype=torch.int32, device=dev)
            gate = torch.full((n * k,), -1.0, dtype=torch.float32, device=dev)
            counts = torch.full((e,), -1, dtype=torch.int32, device=dev)
            offsets = torch.full((e + 1,), -1, dtype=torch.int32, device=dev)
            perm = torch.full((n * k,), -1, dtype=torch.int32, device=dev)
            rc = binding.route_noalloc(x.data_ptr(), wr_dev.data_ptr(), None, c.data_ptr(), n, h, e, k,
                                       stream, ids.data_ptr(), gate.data_ptr(), counts.data_ptr(),
                                       offsets.data_ptr(), perm.data_ptr())
            assert rc == binding.OLED_OK, binding.strerror(rc)
            torch.cuda.synchronize(dev)
            assert np.array_equal(ids.cpu().numpy().reshape(n, k), ref["ids"])
            assert np.array_equal(gate.cpu().numpy().view(np.uint32).reshape(n, k),
                                  ref["gate"].view(np.uint32))            # same kernels: bit-exact
            assert np.array_equal(counts.cpu().numpy(), ref["counts"])
            assert np.array_equal(perm.cpu().numpy(), ref["perm"])
            off = offsets.cpu().numpy()
            assert off[0] == 0 and np.array_equal(np.diff(off), ref["counts"])
            # ... and against the oracle (independent of the CUDA path) on the same input bits
            logits = oracle_moe.gate_logits(oracle_moe.bf16_to_f32(h_bits),
                                            oracle_moe.bf16_to_f32(run.router_bits[0]), None)
            o_ids, o_gate = oracle_moe.topk_route(logits, k)
            o_counts, o_offsets, o_perm, _ = oracle_moe.permutation(o_ids, e)
            assert np.array_equal(ids.cpu().numpy().reshape(n, k), o_ids)
            assert np.array_equal(gate.cpu().numpy().view(np.uint32).reshape(n, k), o_gate.view(np.uint32))
            assert np.array_equal(counts.cpu().numpy(), o_counts)
            assert np.array_equal(off, o_offsets)
            assert np.array_equal(perm.cpu().numpy(), o_perm)
        # beyond the stated maximum: a clear error, nothing launched
        big = binding.NOALLOC_MAX_TOKENS + 1
        rc = binding.route_noalloc(x.data_ptr(), wr_dev.data_ptr(), None, c.data_ptr(), big, h, e, k,
                                   stream, ids.data_ptr(), gate.data_ptr(), counts.data_ptr(),
                                   offsets.data_ptr(), perm.data_ptr())
        assert rc == binding.ERR_TOO_MANY_TOKENS
    finally:
        run.close()
