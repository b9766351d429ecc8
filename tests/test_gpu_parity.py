"""Parity of the CUDA path (through the C ABI) against the CPU oracle on seeded inputs.

Discrete results (expert ids, permutation, counts, integer reuse scores, resident sets,
counters) must match bit for bit; gate scores are fp32 values computed in the same operation
order and must also match bit for bit; the layer output (bf16 on the GPU, fp64 in the oracle)
must satisfy max-abs error <= 2e-2 and relative L2 error <= 1e-2.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import OracleStack  # noqa: E402
from paper_2609_33385_b200 import synth  # noqa: E402

pytestmark = pytest.mark.gpu

MAX_ABS, REL_L2 = 2e-2, 1e-2


def _runner(w, **kw):
    from paper_2609_33385_b200 import build
    build.build()
    from paper_2609_33385_b200.runner import StackRunner
    return StackRunner(w, **kw)


def _oracle_for(run, caps, policy="priority"):
    w = run.w
    st = OracleStack(w.n_layers, w.hidden, w.n_experts, w.top_k, w.intermediate, caps, policy=policy)
    for l in range(w.n_layers):
        st.register_router(l, run.router_bits[l], run.bias[l])
        if getattr(run, "fp8", False):
            st.register_experts_fp8(l, run.layer_blobs(l))
        else:
            st.register_experts(l, run.layer_blobs(l))
    return st


def _check_out(out_bits, ref, what=""):
    got = synth.bf16_bits_to_f32(out_bits).astype(np.float64)
    err = np.abs(got - ref).max() if ref.size else 0.0
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30) if ref.size else 0.0
    assert err <= MAX_ABS and rel <= REL_L2, f"{what}: max-abs {err:.3e}, rel-L2 {rel:.3e}"
    return err, rel


def _check_step(run, layer, n_tokens, out_t, ref, check_out=True):
    from paper_2609_33385_b200.runner import dev_to_bits
    dbg = run.ctx.debug_last(layer, n_tokens)
    e = run.w.n_experts
    assert np.array_equal(dbg["ids"], ref["ids"]), "expert ids differ"
    assert np.array_equal(dbg["gate"].view(np.uint32), ref["gate"].view(np.uint32)), "gate scores differ"
    assert np.array_equal(dbg["counts"], ref["counts"])
    assert np.array_equal(dbg["perm"], ref["perm"]), "permutation differs"
    assert [int(v) for v in dbg["scores"]] == list(ref["scores"]), "reuse scores differ"
    assert set(np.flatnonzero(dbg["resident_before"])) == ref["resident_before"]
    assert set(np.flatnonzero(dbg["resident_after"])) == ref["resident_after"]
    dbp = run.ctx.debug_perm(layer, n_tokens)
    assert np.array_equal(dbp["offsets"], ref["offsets"]), "offsets differ"
    assert np.array_equal(dbp["pos"], ref["pos"]), "inverse permutation differs"
    if n_tokens:
        logits = run.ctx.debug_logits(layer, n_tokens)
        assert np.array_equal(logits.view(np.uint32), ref["logits"].view(np.uint32)), "logits differ"
    if check_out:
        _check_out(dev_to_bits(out_t), ref["out"], f"layer {layer}")
    assert len(dbg["counts"]) == e


def _check_stats(run, ora):
    for l in range(run.w.n_layers):
        a, b = run.ctx.stats(l), ora.stats(l)
        assert (a.steps, a.hits, a.misses, a.bytes_moved, a.evictions, a.active_experts, a.assignments,
                a.fills_reused, a.ideal_hits) == \
               (b.steps, b.hits, b.misses, b.bytes_moved, b.evictions, b.active_experts, b.assignments,
                b.fills_reused, b.ideal_hits)
    a, b = run.ctx.stats(-1), ora.stats(-1)
    assert (a.hits, a.misses, a.bytes_moved) == (b.hits, b.misses, b.bytes_moved)


def _run_stack(run, ora, check_out=True):
    """Replay mode: the oracle is fed the bf16 inputs the GPU saw at every call."""
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = run.w
    dev = run.device
    out = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=dev)
    bufs = [torch.empty_like(out), torch.empty_like(out)]
    for b, i, h_bits, conf in synth.denoise_inputs(w):
        x = bits_to_dev(h_bits, dev)
        c = torch.from_numpy(conf).to(dev)
        for l in range(w.n_layers):
            run.step(l, x, c, out)
            ref = ora.denoise_step(l, dev_to_bits(x), conf)
            _check_step(run, l, w.tokens, out, ref, check_out)
            nxt = bufs[l & 1]
            run.ctx.residual_add(x.data_ptr(), out.data_ptr(), nxt.data_ptr(), x.numel())
            # the residual kernel: bf16(x + out) with one rounding
            exp = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(dev_to_bits(x)) +
                                         synth.bf16_bits_to_f32(dev_to_bits(out)))
            assert np.array_equal(dev_to_bits(nxt), exp)
            x = nxt
    _check_stats(run, ora)


@pytest.mark.parametrize("ffn_impl", [1, 0], ids=["ffn-plain", "ffn-tcgen05"])
def test_tiny_stack_elementwise(ffn_impl):
    w = synth.tiny()
    run = _runner(w, capacity=[3, 5], ffn_impl=ffn_impl)
    try:
        _run_stack(run, _oracle_for(run, [3, 5]))
    finally:
        run.close()


@pytest.mark.parametrize("ffn_impl", [1, 0], ids=["ffn-plain", "ffn-tcgen05"])
def test_config1_full_run(ffn_impl):
    w = synth.config(0)                        # hidden 512, 16 experts top-2, I 1024, 32 tokens
    run = _runner(w, ffn_impl=ffn_impl)
    try:
        _run_stack(run, _oracle_for(run, [w.capacity]))
        st = run.ctx.stats()
        assert st.steps == w.iters and st.misses > 0 and st.hits > 0
    finally:
        run.close()


@pytest.mark.parametrize("n_tokens", [0, 1, 7, 33, 150])
def test_ragged_token_counts(n_tokens):
    """Token counts that leave experts empty, span several 16-row tiles and end in a ragged tail."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=6, top_k=3, hidden=512, intermediate=256)
    run = _runner(w, capacity=[2], max_tokens=160)
    ora = _oracle_for(run, [2])
    try:
        for rep in range(2):
            h_bits, conf = synth.flat_tokens(w, n_tokens, rep)
            x = bits_to_dev(h_bits, run.device) if n_tokens else torch.empty((0, w.hidden), dtype=torch.bfloat16, device=run.device)
            c = torch.from_numpy(conf).to(run.device)
            out = torch.zeros((max(n_tokens, 1), w.hidden), dtype=torch.bfloat16, device=run.device)[:n_tokens]
            run.step(0, x, c, out)
            ref = ora.denoise_step(0, h_bits.reshape(n_tokens, w.hidden), conf)
            _check_step(run, 0, n_tokens, out, ref)
        _check_stats(run, ora)
    finally:
        run.close()


@pytest.mark.parametrize("n_experts,n_tokens", [(64, 5), (64, 200), (64, 310), (128, 33), (128, 256), (128, 300)])
def test_gate_with_64_and_128_experts(n_experts, n_tokens):
    """The expert counts of the benchmark configurations at a small hidden size, with one, two and four
    tokens per CTA of the few-token gate kernel (several passes over the experts per warp): logits,
    ids, gate scores bit for bit; and the two layers as one iteration, whose second gate kernel
    carries the first layer's combine."""
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=2, n_experts=n_experts, top_k=8, hidden=768, intermediate=128)
    run = _runner(w, capacity=[n_experts // 2, n_experts // 2], max_tokens=n_tokens)
    ora = _oracle_for(run, [n_experts // 2, n_experts // 2])
    try:
        h_bits, conf = synth.flat_tokens(w, n_tokens, 3)
        c = torch.from_numpy(conf).to(run.device)
        x = bits_to_dev(h_bits, run.device)
        for layer in range(2):
            out = torch.empty((n_tokens, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(layer, x, c, out)
            ref = ora.denoise_step(layer, dev_to_bits(x), conf)
            _check_step(run, layer, n_tokens, out, ref)
            nxt = torch.empty_like(out)
            run.ctx.residual_add(x.data_ptr(), out.data_ptr(), nxt.data_ptr(), x.numel())
            x = nxt
        # the same two layers as one iteration (the second gate kernel carries the first layer's combine)
        run2 = _runner(w, capacity=[n_experts // 2, n_experts // 2], max_tokens=n_tokens)
        try:
            y = torch.empty((n_tokens, w.hidden), dtype=torch.bfloat16, device=run.device)
            x0 = bits_to_dev(h_bits, run.device)
            run2.ctx.denoise_iteration(x0.data_ptr(), c.data_ptr(), n_tokens, y.data_ptr())
            assert np.array_equal(dev_to_bits(y), dev_to_bits(x))
        finally:
            run2.close()
    finally:
        run.close()


@pytest.mark.parametrize("n", [700, 2100])
def test_many_tokens_per_expert_multi_tile(n):
    """More than 256 rows for one expert: several N tiles per expert in both FFN kernels; the
    larger case also takes the many-token variants of the gate and gather kernels."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=256, intermediate=128)
    run = _runner(w, capacity=[4], max_tokens=n)
    ora = _oracle_for(run, [4])
    try:
        h_bits, conf = synth.flat_tokens(w, n, 7)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)
        ref = ora.denoise_step(0, h_bits, conf)
        assert ref["counts"].max() > 256
        _check_step(run, 0, n, out, ref)
    finally:
        run.close()


@pytest.mark.parametrize("n", [700, 2100])
def test_cta_pair_ffn_form_many_tokens(n):
    """Token tiles of 256 rows with hidden a multiple of 512 and intermediate a multiple of 256: the
    expert FFN runs on CTA pairs (cta_group::2), each CTA holding half of a token tile.  Ragged
    last tiles, several tiles per expert; against the oracle, against the one-CTA form
    (OLED_OPT_FFN_PAIRS 0), which accumulates every output in the same order, and the one-launch
    pair form (gate/up items, then down items behind per-expert counters) against the two-launch
    one (OLED_OPT_FUSE_FFN 0)."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=512, intermediate=256)
    run = _runner(w, capacity=[4], max_tokens=n)
    ora = _oracle_for(run, [4])
    try:
        h_bits, conf = synth.flat_tokens(w, n, 9)
        c = torch.from_numpy(conf).to(run.device)
        ref = ora.denoise_step(0, h_bits, conf)
        assert ref["counts"].max() > 256
        outs = []
        for pairs, fuse in ((1, 1), (0, 1), (1, 0)):   # one launch on pairs; one CTA per tile; two launches on pairs
            run.ctx.set_option(binding.OPT_FFN_PAIRS, pairs)
            run.ctx.set_option(binding.OPT_FUSE_FFN, fuse)
            out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, bits_to_dev(h_bits, run.device), c, out)
            _check_step(run, 0, n, out, ref)
            outs.append(out.float().cpu().numpy().astype(np.float64))
            run.ctx.reset_cache()
        assert np.linalg.norm(outs[0] - outs[1]) <= 1e-3 * np.linalg.norm(outs[1])
        assert np.array_equal(outs[0], outs[2])   # the same items in the same arithmetic, one launch or two
        # token rows gathered by the FFN launch itself (the default where it applies, n = 2100
        # here) or by a gather kernel in front: the same operands
        for fuse in (1, 0):
            run.ctx.set_option(binding.OPT_FFN_PAIRS, 1)
            run.ctx.set_option(binding.OPT_FUSE_FFN, fuse)
            run.ctx.set_option(binding.OPT_GATHER_IN_FFN, 0)
            out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, bits_to_dev(h_bits, run.device), c, out)
            _check_step(run, 0, n, out, ref)
            assert np.array_equal(outs[0], out.float().cpu().numpy().astype(np.float64))
            run.ctx.reset_cache()
    finally:
        run.close()


@pytest.mark.parametrize("hidden", [512, 4608])
def test_gather_in_ffn_with_cache_misses(hidden):
    """A many-token step with misses: the launches over the fetched experts gather their own token rows
    as well (token tile 256 whatever their counts), ragged tiles included.  hidden 4608: a row is moved
    as two pieces (8192 + 1024 bytes)."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    n = 2100
    # (weights scaled with the contraction length, so that the outputs stay of order one)
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=hidden, intermediate=256,
                   weight_std=0.05 * (512 / hidden) ** 0.5)
    run = _runner(w, capacity=[2], max_tokens=n)
    ora = _oracle_for(run, [2])
    try:
        got = []
        for seed in (9, 10):
            h_bits, conf = synth.flat_tokens(w, n, seed)
            ref = ora.denoise_step(0, h_bits, conf)
            out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device), out)
            _check_step(run, 0, n, out, ref)
            got.append(dev_to_bits(out).copy())
        assert run.ctx.stats().misses > 0
        # the same two steps with a gather kernel in front: the same bits
        run.ctx.reset_cache()
        run.ctx.set_option(binding.OPT_GATHER_IN_FFN, 0)
        for i, seed in enumerate((9, 10)):
            h_bits, conf = synth.flat_tokens(w, n, seed)
            out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device), out)
            assert np.array_equal(got[i], dev_to_bits(out))
    finally:
        run.close()


def test_output_bit_identical_at_every_capacity():
    """Offloading is lossless (Sec. 5.1): routing and output do not depend on the capacity."""
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=1, blocks=1, iters=4, n_experts=8, top_k=2)
    outs, miss = [], []
    for cap in (1, 3, 8):
        run = _runner(w, capacity=[cap])
        try:
            res = []
            for _, _, h_bits, conf in synth.denoise_inputs(w):
                x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
                out = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=run.device)
                run.step(0, x, c, out)
                res.append((dev_to_bits(out).copy(), run.ctx.debug_last(0, w.tokens)["ids"].copy()))
            outs.append(res)
            miss.append(run.ctx.stats().misses)
        finally:
            run.close()
    for res in outs[1:]:
        for (o0, i0), (o1, i1) in zip(outs[0], res):
            assert np.array_equal(i0, i1) and np.array_equal(o0, o1)
    assert miss[0] >= miss[1] >= miss[2]


def test_iteration_entry_points_match_layer_by_layer_steps():
    """oled_denoise_iteration (device and host buffers) == steps + residual adds, bit for bit."""
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=3, n_experts=8, top_k=2)
    runs = [_runner(w, capacity=[3, 4, 2]) for _ in range(3)]
    try:
        dev = runs[0].device
        out = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=dev)
        bufs = [torch.empty_like(out), torch.empty_like(out)]
        for _, _, h_bits, conf in synth.denoise_inputs(w):
            x, c = bits_to_dev(h_bits, dev), torch.from_numpy(conf).to(dev)
            ref = dev_to_bits(runs[0].iteration(x, c, bufs, out)).copy()
            y = torch.empty_like(out)
            runs[1].ctx.denoise_iteration(x.data_ptr(), c.data_ptr(), w.tokens, y.data_ptr())
            assert np.array_equal(dev_to_bits(y), ref)
            hx = torch.from_numpy(h_bits.view(np.int16)).pin_memory()
            hc = torch.from_numpy(conf).pin_memory()
            hy = torch.empty((w.tokens, w.hidden), dtype=torch.int16).pin_memory()
            runs[2].ctx.denoise_iteration_host(hx.data_ptr(), hc.data_ptr(), w.tokens, hy.data_ptr())
            assert np.array_equal(hy.numpy().view(np.uint16), ref)
        assert runs[0].ctx.stats() == runs[1].ctx.stats() == runs[2].ctx.stats()
        assert runs[0].ctx.stats().steps == 3 * w.iters * w.blocks
    finally:
        for r in runs:
            r.close()


def test_l2_prefetch_across_layers_changes_no_bit():
    """OLED_OPT_L2_PREFETCH only calls weights into L2: with all experts resident (no miss, so the
    prefetch kernel runs behind every layer; value 2 lifts the stream-length condition the tiny
    shape would not meet) the iterations' outputs and statistics equal those with it off."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=3, n_experts=8, top_k=2)
    runs = [_runner(w, capacity=[8, 8, 8]) for _ in range(2)]
    try:
        runs[0].ctx.set_option(binding.OPT_L2_PREFETCH, 2)
        runs[1].ctx.set_option(binding.OPT_L2_PREFETCH, 0)
        dev = runs[0].device
        for _, _, h_bits, conf in synth.denoise_inputs(w):
            x, c = bits_to_dev(h_bits, dev), torch.from_numpy(conf).to(dev)
            ys = []
            for r in runs:
                y = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=dev)
                r.ctx.denoise_iteration(x.data_ptr(), c.data_ptr(), w.tokens, y.data_ptr())
                ys.append(dev_to_bits(y).copy())
            assert np.array_equal(ys[0], ys[1])
        assert runs[0].ctx.stats() == runs[1].ctx.stats()
        assert runs[0].ctx.launch_count() > runs[1].ctx.launch_count()   # the prefetch kernel did run
    finally:
        for r in runs:
            r.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=1)
    run_d, run_h = _runner(w, capacity=[3]), _runner(w, capacity=[3])
    try:
        for _, _, h_bits, conf in synth.denoise_inputs(w):
            x, c = bits_to_dev(h_bits, run_d.device), torch.from_numpy(conf).to(run_d.device)
            out = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=run_d.device)
            run_d.step(0, x, c, out)
            hx = torch.from_numpy(h_bits.view(np.int16)).pin_memory()
            hc = torch.from_numpy(conf).pin_memory()
            ho = torch.empty((w.tokens, w.hidden), dtype=torch.int16).pin_memory()
            run_h.step_host(0, hx, hc, ho)
            assert np.array_equal(ho.numpy().view(np.uint16), dev_to_bits(out))
        assert run_d.ctx.stats() == run_h.ctx.stats()
    finally:
        run_d.close()
        run_h.close()


def test_errors_are_codes_not_crashes():
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1)
    ctx = binding.OledContext(1, w.hidden, w.n_experts, w.top_k, w.intermediate, 8, [2])
    try:
        x = torch.zeros((8, w.hidden), dtype=torch.bfloat16, device="cuda:0")
        c = torch.zeros(8, device="cuda:0")
        out = torch.zeros_like(x)
        assert ctx.denoise_step_rc(0, x.data_ptr(), c.data_ptr(), 8, out.data_ptr()) == binding.ERR_NOT_REGISTERED
        wr, _ = synth.router_weights(w, 0)
        wr_d = bits_to_dev(wr, "cuda:0")
        ctx.register_router(0, wr_d.data_ptr())
        pageable = torch.zeros((w.n_experts, w.expert_elems), dtype=torch.int16)
        with pytest.raises(binding.OledError) as ei:
            ctx.register_experts(0, pageable.data_ptr(), w.expert_bytes)
        assert ei.value.code == binding.ERR_NOT_PINNED
        pinned = torch.zeros((w.n_experts, w.expert_elems), dtype=torch.int16).pin_memory()
        with pytest.raises(binding.OledError) as ei:
            ctx.register_experts(0, pinned.data_ptr(), w.expert_bytes - 16)
        assert ei.value.code == binding.ERR_INVALID_ARG
        ctx.register_experts(0, pinned.data_ptr(), w.expert_bytes)
        assert ctx.denoise_step_rc(0, x.data_ptr(), c.data_ptr(), 9, out.data_ptr()) == binding.ERR_TOO_MANY_TOKENS
        assert ctx.denoise_step_rc(1, x.data_ptr(), c.data_ptr(), 8, out.data_ptr()) == binding.ERR_INVALID_ARG
        assert ctx.denoise_step_rc(0, x.data_ptr(), c.data_ptr(), 8, x.data_ptr()) == binding.ERR_INVALID_ARG
        assert ctx.denoise_step_rc(0, None, c.data_ptr(), 8, out.data_ptr()) == binding.ERR_INVALID_ARG
        # rows are moved with 16-byte vector accesses: a view that starts inside one is refused
        big = torch.zeros(8 * w.hidden + 8, dtype=torch.bfloat16, device="cuda:0")
        assert ctx.denoise_step_rc(0, big[4:].data_ptr(), c.data_ptr(), 8, out.data_ptr()) == binding.ERR_INVALID_ARG
        assert ctx.denoise_step_rc(0, x.data_ptr(), c.data_ptr(), 8, big[4:].data_ptr()) == binding.ERR_INVALID_ARG
        assert ctx.denoise_step_rc(0, x.data_ptr(), c.data_ptr(), 8, out.data_ptr()) == binding.OLED_OK
        ctx.synchronize()
        assert float(out.float().abs().max()) == 0.0          # zero weights -> zero output
        with pytest.raises(binding.OledError):
            binding.OledContext(1, 250, 8, 2, 128, 8, [2])     # hidden not a multiple of 256
        with pytest.raises(binding.OledError):
            binding.OledContext(1, 256, 8, 2, 128, 8, [9])     # capacity > E
    finally:
        ctx.destroy()


def test_reset_cache_returns_to_cold_state():
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1)
    run = _runner(w, capacity=[w.n_experts])
    try:
        h_bits, conf = synth.flat_tokens(w, 5)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((5, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)
        m1 = run.ctx.stats().misses
        run.step(0, x, c, out)
        assert run.ctx.stats().misses == m1 and m1 > 0        # second identical step: all hits
        run.ctx.reset_cache()
        assert run.ctx.stats().steps == 0
        run.step(0, x, c, out)
        assert run.ctx.stats().misses == m1
    finally:
        run.close()


@pytest.mark.parametrize("policy", ["lru", "lfu"])
def test_comparison_policies_match_oracle(policy):
    """LRU / LFU retention through the real step: resident sets, counters and outputs."""
    w = synth.tiny(n_layers=2, blocks=2, iters=4, n_experts=8, top_k=2)
    run = _runner(w, capacity=[3, 2], policy=policy)
    try:
        _run_stack(run, _oracle_for(run, [3, 2], policy=policy))
    finally:
        run.close()


def test_layer_adaptive_sizing_through_the_iteration_entry_point():
    """oled_denoise_iteration with a refresh period of 2: capacities, resident sets and counters
    follow the oracle's layer-adaptive sizing; outputs stay within tolerance."""
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=3, blocks=3, iters=3, n_experts=8, top_k=2)
    caps = [3, 3, 3]
    run = _runner(w, capacity=caps, adapt_period=2, staging_slots=8)
    ora = _oracle_for(run, caps)
    try:
        dev = run.device
        y = torch.empty((w.tokens, w.hidden), dtype=torch.bfloat16, device=dev)
        out = torch.empty_like(y)
        bufs = [torch.empty_like(y), torch.empty_like(y)]
        shadow = _runner(w, capacity=caps, staging_slots=8)       # same inputs, step by step, for replay
        changed = False
        for it, (_, _, h_bits, conf) in enumerate(synth.denoise_inputs(w)):
            x, c = bits_to_dev(h_bits, dev), torch.from_numpy(conf).to(dev)
            run.ctx.denoise_iteration(x.data_ptr(), c.data_ptr(), w.tokens, y.data_ptr())
            # replay the same iteration layer by layer on the shadow context to feed the oracle
            xs = x
            for l in range(w.n_layers):
                shadow.step(l, xs, c, out)
                ora.denoise_step(l, dev_to_bits(xs), conf)
                nxt = bufs[l & 1]
                shadow.ctx.residual_add(xs.data_ptr(), out.data_ptr(), nxt.data_ptr(), xs.numel())
                xs = nxt
            assert np.array_equal(dev_to_bits(y), dev_to_bits(xs))   # capacity never changes outputs
            if (it + 1) % 2 == 0:
                want = ora.adapt_capacity()
                assert run.ctx.get_capacity() == want and sum(want) == sum(caps)
                changed = changed or want != caps
            for l in range(w.n_layers):
                a, b = run.ctx.stats(l), ora.stats(l)
                assert (a.hits, a.misses, a.evictions, a.fills_reused) == \
                       (b.hits, b.misses, b.evictions, b.fills_reused), (it, l)
        assert changed, "the allocation never moved: the test exercises nothing"
        shadow.close()
    finally:
        run.close()


def test_bounded_device_wait_reports_timeout_and_context_survives():
    """Failure path without a fault: the FFN kernels' load producers are told to issue nothing, so
    the consumers' bounded waits run out; the kernels flag it and return, the host reads
    OLED_ERR_TIMEOUT, and after oled_clear_status() the same context computes correct results."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=1)
    run = _runner(w, capacity=[w.n_experts])
    ora = _oracle_for(run, [w.n_experts])
    try:
        h_bits, conf = synth.flat_tokens(w, 5)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((5, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)                                   # warm: everything resident
        ref = ora.denoise_step(0, h_bits, conf)
        run.ctx.synchronize()
        run.ctx.set_option(binding.OPT_TEST_WITHHOLD_LOADS, 1)
        run.step(0, x, c, out)                                   # hits only: one FFN launch pair
        assert run.ctx.synchronize_rc() == binding.ERR_TIMEOUT
        assert run.ctx.synchronize_rc() == binding.ERR_TIMEOUT   # sticky until cleared
        run.ctx.set_option(binding.OPT_TEST_WITHHOLD_LOADS, 0)
        run.ctx.clear_status()
        assert run.ctx.synchronize_rc() == binding.OLED_OK
        ora.denoise_step(0, h_bits, conf)                        # keep the oracle's counters in step
        run.step(0, x, c, out)
        _check_out(dev_to_bits(out), ora.denoise_step(0, h_bits, conf)["out"])
        ns, runs = run.ctx.policy_time()
        assert runs == 3 and ns > 0
    finally:
        run.close()


def test_bounded_device_wait_in_the_cta_pair_kernel():
    """The same failure path in the many-token FFN on CTA pairs: no item is ever published, the
    bounded waits of every role of both CTAs run out, the cluster's kernels return, the host
    reads OLED_ERR_TIMEOUT, and afterwards the same context is in parity again."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=512, intermediate=256)
    n = 700
    run = _runner(w, capacity=[4], max_tokens=n)
    ora = _oracle_for(run, [4])
    try:
        h_bits, conf = synth.flat_tokens(w, n, 11)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)                                   # warm: everything resident
        ref = ora.denoise_step(0, h_bits, conf)
        assert ref["counts"].max() > 256                         # token tiles of 256 rows: the pair kernel
        _check_out(dev_to_bits(out), ref["out"])
        run.ctx.set_option(binding.OPT_TEST_WITHHOLD_LOADS, 1)
        run.step(0, x, c, out)
        assert run.ctx.synchronize_rc() == binding.ERR_TIMEOUT
        run.ctx.set_option(binding.OPT_TEST_WITHHOLD_LOADS, 0)
        run.ctx.clear_status()
        assert run.ctx.synchronize_rc() == binding.OLED_OK
        ora.denoise_step(0, h_bits, conf)                        # keep the oracle's counters in step
        run.step(0, x, c, out)
        _check_out(dev_to_bits(out), ora.denoise_step(0, h_bits, conf)["out"])
    finally:
        run.close()


def test_self_check_is_silent_on_valid_steps_and_flags_a_corrupted_permutation():
    """OLED_OPT_SELF_CHECK: the checking kernels find nothing on valid steps (parity unchanged, guard
    words intact); with the first two sorted rows exchanged by the test aid - both still valid
    rows, so nothing faults - the next synchronising call returns OLED_ERR_SELF_CHECK and the
    report names the broken invariant; after oled_clear_status() the context is in parity again."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(blocks=1, iters=3)
    run = _runner(w, capacity=[3, 5], max_tokens=max(w.tokens, 9))
    ora = _oracle_for(run, [3, 5])
    try:
        run.ctx.set_option(binding.OPT_SELF_CHECK, 1)
        _run_stack(run, ora)                                     # every step checked, all in parity
        run.ctx.synchronize()
        assert run.ctx.self_check_report() == ([], -1, 0)
        h_bits, conf = synth.flat_tokens(w, 9, 3)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((9, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.ctx.set_option(binding.OPT_TEST_CORRUPT_PERM, 1)
        run.step(0, x, c, out)
        ora.denoise_step(0, h_bits, conf)                        # keep the oracle's cache state in step
        assert run.ctx.synchronize_rc() == binding.ERR_SELF_CHECK
        names, index, guard = run.ctx.self_check_report()
        assert "inverse" in names and index in (0, 1) and guard == 0
        assert run.ctx.synchronize_rc() == binding.ERR_SELF_CHECK   # sticky until cleared
        run.ctx.set_option(binding.OPT_TEST_CORRUPT_PERM, 0)
        run.ctx.clear_status()
        assert run.ctx.synchronize_rc() == binding.OLED_OK
        run.step(0, x, c, out)
        _check_step(run, 0, 9, out, ora.denoise_step(0, h_bits, conf))
        assert run.ctx.self_check_report() == ([], -1, 0)
    finally:
        run.close()


def test_maximum_expert_count_and_top_k():
    """512 experts (OLED_MAX_EXPERTS) with top-32 (OLED_MAX_TOPK): the widest gate the ABI allows."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=512, top_k=32, hidden=256, intermediate=128)
    run = _runner(w, capacity=[40], max_tokens=8)
    ora = _oracle_for(run, [40])
    try:
        for rep, n in enumerate((3, 8)):
            h_bits, conf = synth.flat_tokens(w, n, 20 + rep)
            x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
            out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, x, c, out)
            _check_step(run, 0, n, out, ora.denoise_step(0, h_bits, conf))
        _check_stats(run, ora)
    finally:
        run.close()


def test_degenerate_routing_cases():
    """Identical tokens (one expert set takes every token), zero confidences (all reuse scores
    zero: retention falls back to the id order) and top-k equal to the number of experts."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=4, top_k=4, hidden=256, intermediate=128)
    run = _runner(w, capacity=[2], max_tokens=40)
    ora = _oracle_for(run, [2])
    try:
        h_bits, conf = synth.flat_tokens(w, 40, 30)
        same = np.repeat(h_bits[:1], 40, axis=0)                       # every token identical
        zero_c = np.zeros(40, np.float32)
        for hb, cf in ((same, conf), (h_bits, zero_c), (same, zero_c)):
            x, c = bits_to_dev(hb, run.device), torch.from_numpy(cf).to(run.device)
            out = torch.empty((40, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, x, c, out)
            ref = ora.denoise_step(0, hb, cf)
            _check_step(run, 0, 40, out, ref)
            assert ref["counts"].tolist() == [40, 40, 40, 40]           # k = E: every expert, every token
        _check_stats(run, ora)
    finally:
        run.close()
    # a single expert set for all tokens with k < E: two experts hold all 2*T assignments
    w2 = synth.tiny(n_layers=1, n_experts=8, top_k=2, hidden=256, intermediate=128)
    run = _runner(w2, capacity=[3], max_tokens=300)
    ora = _oracle_for(run, [3])
    try:
        h_bits, conf = synth.flat_tokens(w2, 300, 31)
        same = np.repeat(h_bits[:1], 300, axis=0)
        x, c = bits_to_dev(same, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((300, w2.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)
        ref = ora.denoise_step(0, same, conf)
        assert sorted(ref["counts"].tolist())[-2:] == [300, 300] and ref["counts"].sum() == 600
        _check_step(run, 0, 300, out, ref)
    finally:
        run.close()


def test_non_finite_activations_keep_routing_defined_and_the_context_usable():
    """NaN and Inf in the hidden states: a NaN logit ranks as -inf, so the k ids of every token
    stay distinct and all discrete results still match the oracle; rows of clean tokens are
    unaffected; the next clean step is in full parity."""
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=1)
    run = _runner(w, capacity=[3], max_tokens=40)
    ora = _oracle_for(run, [3])
    try:
        h_bits, conf = synth.flat_tokens(w, 40, 77)
        bad = h_bits.copy()
        bad[3, :] = 0x7FC0      # a whole NaN row
        bad[5, 17] = 0x7FC0     # one NaN element
        bad[7, 1] = 0x7F80      # +Inf
        bad[9, 2] = 0xFF80      # -Inf
        x, c = bits_to_dev(bad, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((40, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)
        with np.errstate(all="ignore"):
            ref = ora.denoise_step(0, bad, conf)
        dbg = run.ctx.debug_last(0, 40)
        assert np.array_equal(dbg["ids"], ref["ids"])
        assert all(len(set(row)) == w.top_k for row in dbg["ids"].tolist())
        assert np.array_equal(np.isnan(dbg["gate"]), np.isnan(ref["gate"]))
        ok = ~np.isnan(ref["gate"])
        assert np.array_equal(dbg["gate"][ok].view(np.uint32), ref["gate"][ok].view(np.uint32))
        assert np.array_equal(dbg["counts"], ref["counts"]) and np.array_equal(dbg["perm"], ref["perm"])
        assert [int(v) for v in dbg["scores"]] == list(ref["scores"])
        assert set(np.flatnonzero(dbg["resident_after"])) == ref["resident_after"]
        clean = [t for t in range(40) if t not in (3, 5, 7, 9)]
        _check_out(dev_to_bits(out)[clean], ref["out"][clean], "clean rows")
        x2 = bits_to_dev(h_bits, run.device)
        run.step(0, x2, c, out)
        _check_step(run, 0, 40, out, ora.denoise_step(0, h_bits, conf))
        _check_stats(run, ora)
    finally:
        run.close()


def test_fp8_expert_store_tiny_stack():
    """fp8 (e4m3 + row scales) expert blobs: same discrete results, outputs within the same
    tolerance of the oracle evaluated on the dequantised weights, half the bytes moved."""
    w = synth.tiny(blocks=2, iters=3)
    run = _runner(w, capacity=[3, 5], fp8=True)
    try:
        ora = _oracle_for(run, [3, 5])
        _run_stack(run, ora)
        st = run.ctx.stats()
        assert st.bytes_moved == st.misses * synth.fp8_blob_bytes(w)
        assert synth.fp8_blob_bytes(w) < 0.55 * w.expert_bytes
    finally:
        run.close()


@pytest.mark.parametrize("n", [40, 300, 700])
def test_fp8_expert_store_token_tile_variants(n):
    """fp8 blobs through every FFN tile form that exists for them: stacked (token tiles up to 32
    rows) and two accumulators (64 and 128 rows; fp8 stores stop at 128-row tiles, so the
    700-token case takes several tiles per expert)."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=512, intermediate=256)
    run = _runner(w, capacity=[4], max_tokens=n, fp8=True)
    ora = _oracle_for(run, [4])
    try:
        h_bits, conf = synth.flat_tokens(w, n, 50)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)
        _check_step(run, 0, n, out, ora.denoise_step(0, h_bits, conf))
    finally:
        run.close()


def test_fp8_direct_form_agrees_with_widening_form_on_wide_range_rows():
    """Token tiles of at most 32 rows take the form whose MMAs read the e4m3 codes directly, the
    token rows entering as two e4m3 terms after a per-row power-of-two scale.  Rows with a wide
    dynamic range (elements 2^-12 below the row's maximum), an all-zero row and a row 2^10 larger
    than the rest: same discrete results, outputs within tolerance of the oracle, and the two
    forms (OLED_OPT_FP8_DIRECT 1 / 0) agree far more closely than either has to with the oracle."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=512, intermediate=256)
    n = 24
    run = _runner(w, capacity=[4], max_tokens=n, fp8=True)
    ora = _oracle_for(run, [4])
    try:
        h_bits, conf = synth.flat_tokens(w, n, 51)
        f = (h_bits.astype(np.uint32) << 16).view(np.float32).copy()
        f[:, ::3] *= 2.0 ** -12          # a third of every row far below the row's maximum
        f[3, :] = 0.0                    # an all-zero row
        f[5, :] *= 2.0 ** 10             # one row far above the others
        h_bits = (f.view(np.uint32) >> 16).astype(np.uint16)   # (scaling by powers of two is exact in bf16)
        c = torch.from_numpy(conf).to(run.device)
        with np.errstate(over="ignore"):   # exp(-a) of the large row's gate values overflows to inf: silu -> -0
            ref = ora.denoise_step(0, h_bits, conf)
        outs = []
        for direct in (1, 0):
            run.ctx.set_option(binding.OPT_FP8_DIRECT, direct)
            out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
            run.step(0, bits_to_dev(h_bits, run.device), c, out)
            if direct:
                _check_step(run, 0, n, out, ref, check_out=False)
            outs.append(out.float().cpu().numpy().astype(np.float64))
            run.ctx.reset_cache()
        a, b = outs
        assert np.all(a[3] == 0.0) and np.all(b[3] == 0.0) and np.all(ref["out"][3] == 0.0)
        for t in range(n):   # row by row and relative: the rows differ in scale by orders of magnitude
            den = np.linalg.norm(ref["out"][t])
            if den > 0:
                assert np.linalg.norm(a[t] - ref["out"][t]) / den <= REL_L2, ("direct form against the oracle", t)
                assert np.linalg.norm(b[t] - ref["out"][t]) / den <= REL_L2, ("widening form against the oracle", t)
                assert np.linalg.norm(a[t] - b[t]) / den < 3e-3, ("the two forms", t)
    finally:
        run.close()


def test_fp8_direct_form_takes_several_token_tiles_per_expert():
    """After a step in which no expert received more than 16 rows, the direct fp8 form's hit launch
    uses 16-row token tiles; a following step that sends all 24 tokens to the same two experts
    then needs two tiles per expert (the second one ragged)."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=8, top_k=2, hidden=256, intermediate=128)
    n = 24
    run = _runner(w, capacity=[8], max_tokens=n, fp8=True)
    ora = _oracle_for(run, [8])
    try:
        h_bits, conf = synth.flat_tokens(w, n, 52)
        same = np.repeat(h_bits[:1], n, axis=0)                  # every token the same row: one routing decision
        c = torch.from_numpy(conf).to(run.device)
        out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
        for rep, bits in enumerate((h_bits, h_bits, same, h_bits)):
            run.step(0, bits_to_dev(bits, run.device), c, out)
            ref = ora.denoise_step(0, bits, conf)
            if rep < 2:
                assert ref["counts"].max() <= 16
            if rep == 2:
                assert sorted(ref["counts"])[-2:] == [n, n]
            _check_step(run, 0, n, out, ref)
    finally:
        run.close()


def test_fp8_subnormal_codes_decode_exactly():
    """Blobs whose row scales are so large that every code is an e4m3 subnormal (exponent field
    0): the on-chip widening must reproduce them exactly, not flush them."""
    from paper_2609_33385_b200.runner import bits_to_dev
    w = synth.tiny(n_layers=1, n_experts=4, top_k=2, hidden=256, intermediate=128)
    run = _runner(w, capacity=[4], max_tokens=24, fp8=True)
    try:
        h, i = w.hidden, w.intermediate
        rng = np.random.default_rng(77)
        for e in range(w.n_experts):
            blob = run.blobs[0][e]
            codes = (rng.integers(0, 8, size=3 * h * i).astype(np.uint8) |
                     (rng.integers(0, 2, size=3 * h * i).astype(np.uint8) << 7))     # +-{0..7} * 2^-9
            blob[:3 * h * i] = codes
            scales = rng.uniform(2.0, 6.0, size=2 * i + h).astype(np.float32)
            blob[3 * h * i:3 * h * i + 4 * scales.size] = scales.view(np.uint8)
        ora = _oracle_for(run, [4])
        h_bits, conf = synth.flat_tokens(w, 24, 60)
        x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
        out = torch.empty((24, h), dtype=torch.bfloat16, device=run.device)
        run.step(0, x, c, out)
        ref = ora.denoise_step(0, h_bits, conf)
        assert np.abs(ref["out"]).max() > 1e-3                 # the subnormal codes carry the whole signal
        _check_step(run, 0, 24, out, ref)
    finally:
        run.close()


def test_one_launch_and_two_launch_ffn_forms_agree_bit_for_bit():
    """OLED_OPT_FUSE_FFN: gate/up + down projection as one launch (down items wait on per-expert
    completion counters) or as two launches.  Which kernel computes an item does not change its
    arithmetic, so the layer outputs must be bit-identical, and both in parity with the oracle;
    block sizes with one and with two token tiles per expert, cold start so that launches of
    fetched experts (behind event waits) are covered too."""
    from paper_2609_33385_b200 import binding
    from paper_2609_33385_b200.runner import bits_to_dev, dev_to_bits
    w = synth.tiny(n_layers=1, n_experts=6, top_k=3, hidden=512, intermediate=256)
    outs = {}
    for mode in (0, 2):
        run = _runner(w, capacity=[3], max_tokens=160)
        run.ctx.set_option(binding.OPT_FUSE_FFN, mode)
        ora = _oracle_for(run, [3])
        try:
            res = []
            for rep, n in enumerate((7, 33, 60, 150)):      # 150 tokens: 64-row tiles, always two launches
                h_bits, conf = synth.flat_tokens(w, n, 80 + rep)
                x, c = bits_to_dev(h_bits, run.device), torch.from_numpy(conf).to(run.device)
                out = torch.empty((n, w.hidden), dtype=torch.bfloat16, device=run.device)
                run.step(0, x, c, out)
                _check_step(run, 0, n, out, ora.denoise_step(0, h_bits, conf))
                res.append(dev_to_bits(out).copy())
            outs[mode] = res
            _check_stats(run, ora)
        finally:
            run.close()
    for a, b in zip(outs[0], outs[2]):
        assert np.array_equal(a, b)
