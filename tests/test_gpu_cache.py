"""GPU parity of the expert cache: experts staged from pinned host memory into HBM slots on a
copy stream, used by the routed forward on a compute stream.  Checks (i) data: the forward on
cached experts matches the CPU checker within the output bar, and bit-for-bit the forward on the
same experts resident in ordinary device memory; (ii) bookkeeping: slots, evictions and counters
equal the plain model's, operation by operation (integer work: exact)."""
import numpy as np
import pytest
import torch

import oracle
from oracle.cache_sim import ExpertBufferModel, rank_experts
from paper_2308_14352_b200 import binding as B, inputs, layer
from tests.helpers import oracle_pack_layer, output_tolerance, rel_to_max

pytestmark = pytest.mark.gpu


class HostExperts:
    """Packed experts of a small stack in pinned host memory."""

    def __init__(self, shape, n_layers, bits_of_layer, seed):
        self.shape, self.n_layers = shape, n_layers
        self.bits, self.packed, self.scales, self.pin = [], [], [], []
        for l in range(n_layers):
            W = inputs.expert_set(seed, l, shape, 0.02)
            bits = bits_of_layer(l)
            packed, scales = oracle_pack_layer(W, shape, bits)
            self.bits.append(bits)
            self.packed.append(packed)
            self.scales.append(scales)
            pins = []
            for e in range(shape.n_experts):
                pm = [torch.from_numpy(np.ascontiguousarray(p)).pin_memory() for p in packed[e]]
                sdt = np.float16 if shape.scale_dtype == "f16" else np.float32
                sm = [torch.from_numpy(np.ascontiguousarray(s.astype(sdt))).pin_memory() for s in scales[e]]
                pins.append((pm, sm))
            self.pin.append(pins)

    def expert_id(self, l, e):
        return 100 * l + e

    def nbytes(self, l, e):
        pm, sm = self.pin[l][e]
        nb = [t.numel() * t.element_size() for t in pm] + [0] * (3 - len(pm))
        nb += [t.numel() * t.element_size() for t in sm] + [0] * (3 - len(sm))
        return nb

    def register_all(self, ctx, model):
        for l in range(self.n_layers):
            for e in range(self.shape.n_experts):
                pm, sm = self.pin[l][e]
                hp = [t.data_ptr() for t in pm] + [0] * (3 - len(pm))
                hs = [t.data_ptr() for t in sm] + [0] * (3 - len(sm))
                nb = self.nbytes(l, e)
                B.emoe_register_expert(ctx, self.expert_id(l, e), l, self.bits[l][e], hp, hs, nb)
                model.register(self.expert_id(l, e), l, sum(nb))

    def slot_bytes(self):
        return max(sum((b + 255) // 256 * 256 for b in self.nbytes(l, e))
                   for l in range(self.n_layers) for e in range(self.shape.n_experts))


def _bookkeeping(stats):
    """The counters the bookkeeping model has (the library adds its timing fields)."""
    return {k: v for k, v in stats.items() if k not in ("exposed_copy_ns", "timed_acquires")}


def _table_from(acquired, ids_active, bits):
    """Expert table of a layer: acquired pointers for the activated experts; the other entries
    (never touched by the kernels) borrow the pointers of the first activated one."""
    by_e = {e: acquired[i] for i, e in enumerate(ids_active)}
    first = acquired[0]
    entries = []
    for e, b in enumerate(bits):
        src = by_e.get(e, first)
        if e not in by_e:
            b = bits[ids_active[0]]      # a borrowed entry carries the width of the expert it borrows from
        entries.append((b, [src.packed[m] for m in range(3) if src.packed[m]], [src.scales[m] for m in range(3) if src.scales[m]]))
    return B.make_expert_table(entries)


@pytest.mark.parametrize("rule,code", [("forward", B.EVICT_FORWARD), ("lru", B.EVICT_LRU)])
def test_cached_forward_matches_checker_and_model(rule, code):
    shape = inputs.LayerShape(512, 1024, 4, 2, "relu", "softmax_renorm", 128, "f16", "bf16")
    n_layers, T, n_slots = 3, 6, 5
    host = HostExperts(shape, n_layers, lambda l: [[8, 4, 2, 4], [2, 8, 4, 4], [4, 2, 8, 2]][l], seed=31)
    rng = np.random.default_rng(31)
    prior = rng.random((4, 4)).astype(np.float32)
    desc = layer.make_desc(shape)
    dev = torch.device("cuda", 0)
    torch.zeros(1, device=dev)
    ctx = B.emoe_create(0, B.emoe_workspace_bytes(desc, T))
    compute, copy = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    model = ExpertBufferModel(n_slots, n_layers, rule)
    try:
        B.emoe_cache_create(ctx, n_slots, host.slot_bytes(), n_layers, code)
        host.register_all(ctx, model)
        worst = 0.0
        for step in range(4):
            prev_active = None
            for l in range(n_layers):
                x = inputs.activations(31, l, T, shape.d_model, "bf16", batch_tag=step)
                Wr = inputs.router_weight(31, l, shape.d_model, shape.n_experts, std=0.05)
                ids, gates, _ = oracle.route(x, Wr, None, shape.top_k, True)
                active = sorted(set(ids.reshape(-1).tolist()))
                eids = [host.expert_id(l, e) for e in active]
                acq = B.emoe_cache_acquire(ctx, eids, l, compute.cuda_stream, copy.cuda_stream)
                for e, eid in zip(active, eids):
                    s_ref, _, _ = model.acquire(eid, l)
                    assert B.emoe_cache_slot_of(ctx, eid) == s_ref
                # the next layer's likely experts are staged while this layer computes
                nxt = (l + 1) % n_layers
                order = B.emoe_rank_experts(prior, np.array(active, dtype=np.int32))
                assert order.tolist() == rank_experts(prior.tolist(), active)
                pre = [host.expert_id(nxt, int(e)) for e in order[:2]]
                B.emoe_prefetch_experts(ctx, pre, l, copy.cuda_stream)
                for eid in pre:
                    model.prefetch(eid, l)
                table = _table_from(acq, active, host.bits[l])
                xd = torch.from_numpy(x).to(dev).to(torch.bfloat16)
                idd = torch.from_numpy(ids.astype(np.int32)).to(dev)
                gd = torch.from_numpy(gates.astype(np.float32)).to(dev)
                y = torch.empty(T, shape.d_model, dtype=torch.float32, device=dev)
                compute.wait_stream(torch.cuda.current_stream(dev))
                B.emoe_moe_forward_routed(ctx, desc, xd.data_ptr(), T, idd.data_ptr(), gd.data_ptr(), table, y.data_ptr(), None,
                                          compute.cuda_stream)
                B.emoe_cache_release(ctx, eids, compute.cuda_stream)
                for eid in eids:
                    model.release(eid)
                compute.synchronize()
                assert B.emoe_device_status(ctx, compute.cuda_stream) == B.OK
                y_ref = oracle.moe_ffn_combine(x, shape.d_ff, shape.act, shape.group, True, host.bits[l], host.packed[l],
                                               host.scales[l], ids, gates)
                worst = max(worst, rel_to_max(y.cpu().numpy(), y_ref))
                for ll in range(n_layers):
                    for e in range(shape.n_experts):
                        eid = host.expert_id(ll, e)
                        assert B.emoe_cache_slot_of(ctx, eid) == model.where.get(eid, -1)
                assert _bookkeeping(B.emoe_cache_get_stats(ctx)) == model.counters
                prev_active = active
        assert worst <= output_tolerance("bf16"), worst
        st = B.emoe_cache_get_stats(ctx)
        assert st["evictions"] > 0 and st["prefetched"] > 0 and st["hits"] > 0
    finally:
        torch.cuda.synchronize()
        B.emoe_destroy(ctx)


def test_slot_reuse_waits_for_its_reader_and_results_equal_resident_experts():
    """Two slots, three experts: the load that evicts an expert is enqueued right after the
    forward that reads it.  Both forwards must equal, bit for bit, the forwards on the same
    experts kept in ordinary device memory."""
    shape = inputs.LayerShape(768, 3072, 3, 1, "relu", "softmax", 128, "f16", "bf16")
    T = 64
    host = HostExperts(shape, 1, lambda l: [8, 4, 2], seed=33)
    desc = layer.make_desc(shape)
    dev = torch.device("cuda", 0)
    x = inputs.activations(33, 0, T, shape.d_model, "bf16")
    xd = torch.from_numpy(x).to(dev).to(torch.bfloat16)
    gates = np.ones((T, 1), dtype=np.float32)
    gd = torch.from_numpy(gates).to(dev)
    rounds = [np.array([[0], [1]] * (T // 2), dtype=np.int32), np.array([[2], [1]] * (T // 2), dtype=np.int32)]

    # reference: all three experts resident
    with layer.MoELayer(shape, host.bits[0], max_tokens=T) as moe:
        for e in range(3):
            for m in range(2):
                moe.packed[e][m].copy_(host.pin[0][e][0][m].reshape(-1))
                moe.scales[e][m].copy_(host.pin[0][e][1][m].reshape(-1))
        want = [moe.forward_routed(x, ids, gates)[0] for ids in rounds]

    ctx = B.emoe_create(0, B.emoe_workspace_bytes(desc, T))
    compute, copy = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    model = ExpertBufferModel(2, 1, "forward")
    try:
        B.emoe_cache_create(ctx, 2, host.slot_bytes(), 1, B.EVICT_FORWARD)
        host.register_all(ctx, model)
        got = []
        compute.wait_stream(torch.cuda.current_stream(dev))
        for r, ids in enumerate(rounds):
            active = sorted(set(ids.reshape(-1).tolist()))
            eids = [host.expert_id(0, e) for e in active]
            acq = B.emoe_cache_acquire(ctx, eids, 0, compute.cuda_stream, copy.cuda_stream)
            table = _table_from(acq, active, host.bits[0])
            idd = torch.from_numpy(ids).to(dev)
            y = torch.empty(T, shape.d_model, dtype=torch.float32, device=dev)
            compute.wait_stream(torch.cuda.current_stream(dev))
            B.emoe_moe_forward_routed(ctx, desc, xd.data_ptr(), T, idd.data_ptr(), gd.data_ptr(), table, y.data_ptr(), None,
                                      compute.cuda_stream)
            B.emoe_cache_release(ctx, eids, compute.cuda_stream)   # no host synchronisation between the rounds
            got.append(y)
        compute.synchronize()
        assert B.emoe_device_status(ctx, compute.cuda_stream) == B.OK
        for y, w in zip(got, want):
            assert np.array_equal(y.cpu().numpy(), w)
        st = B.emoe_cache_get_stats(ctx)
        assert st["misses"] == 3 and st["hits"] == 1 and st["evictions"] == 1
    finally:
        torch.cuda.synchronize()
        B.emoe_destroy(ctx)


def test_cache_argument_errors():
    shape = inputs.LayerShape(512, 1024, 2, 1, "relu", "softmax", 128, "f16", "bf16")
    desc = layer.make_desc(shape)
    torch.zeros(1, device="cuda:0")
    ctx = B.emoe_create(0, B.emoe_workspace_bytes(desc, 4))
    try:
        with pytest.raises(B.EmoeError):
            B.emoe_prefetch_experts(ctx, [1], 0, 0)                 # no cache yet
        B.emoe_cache_create(ctx, 1, 1 << 20, 2, B.EVICT_FORWARD)
        with pytest.raises(B.EmoeError):
            B.emoe_cache_create(ctx, 1, 1 << 20, 2, B.EVICT_FORWARD)  # one cache per context
        buf = torch.zeros(4096, dtype=torch.uint8).pin_memory()
        with pytest.raises(B.EmoeError) as ei:
            B.emoe_register_expert(ctx, 7, 0, 3, [buf.data_ptr(), 0, 0], [buf.data_ptr(), 0, 0], [1024, 0, 0, 64, 0, 0])
        assert ei.value.status == B.ERR_UNSUPPORTED
        with pytest.raises(B.EmoeError):
            B.emoe_register_expert(ctx, 7, 0, 4, [buf.data_ptr(), 0, 0], [buf.data_ptr(), 0, 0], [2 << 20, 0, 0, 64, 0, 0])  # too big for a slot
        B.emoe_register_expert(ctx, 7, 0, 4, [buf.data_ptr(), 0, 0], [buf.data_ptr() + 2048, 0, 0], [1024, 0, 0, 64, 0, 0])
        B.emoe_register_expert(ctx, 8, 1, 4, [buf.data_ptr(), 0, 0], [buf.data_ptr() + 2048, 0, 0], [1024, 0, 0, 64, 0, 0])
        with pytest.raises(B.EmoeError):
            B.emoe_prefetch_experts(ctx, [9], 0, 0)                 # unknown id
        B.emoe_cache_acquire(ctx, [7], 0, 0, 0)
        with pytest.raises(B.EmoeError) as ei:
            B.emoe_cache_acquire(ctx, [8], 1, 0, 0)                 # the only slot is in use
        assert ei.value.status == B.ERR_CACHE_FULL
        B.emoe_cache_release(ctx, [7], 0)
        B.emoe_cache_acquire(ctx, [8], 1, 0, 0)
        B.emoe_cache_release(ctx, [8], 0)
        # a list that does not fit fails as a whole: the expert it had already taken is let go again
        with pytest.raises(B.EmoeError) as ei:
            B.emoe_cache_acquire(ctx, [7, 8], 0, 0, 0)
        assert ei.value.status == B.ERR_CACHE_FULL
        B.emoe_cache_acquire(ctx, [8], 1, 0, 0)                     # the only slot is free for it
        B.emoe_cache_release(ctx, [8], 0)
        with pytest.raises(B.EmoeError):
            B.emoe_cache_release(ctx, [7, 8], 0)                    # neither is held
    finally:
        torch.cuda.synchronize()
        B.emoe_destroy(ctx)


def test_cached_stack_two_layers_at_the_mixtral_shape():
    """The cached pipeline at the full layer shape (two layers of the Mixtral-like stack): a
    2048-token prefill, then single-token decode steps.  Weights are drawn on the device by the
    stack's seeded generator; the checker packs the same matrices itself (compared byte for byte
    with what the stack staged in host memory) and evaluates sampled outputs."""
    from paper_2308_14352_b200.cached_stack import CachedStack

    w = inputs.WORKLOADS["mixtral_stack_cached"]
    sh, bits = w.shape, list(w.fixed_bits)
    T = 2048
    stack = CachedStack(sh, 2, bits, n_slots=12, max_tokens=T, seed=w.seed)
    try:
        def oracle_expert(l, e):
            ps = [oracle.pack_expert(stack.draw_matrix(l, e, m).cpu().numpy(), bits[e], sh.group, sh.scale_dtype)
                  for m in range(sh.n_matrices)]
            for m, (p, s_) in enumerate(ps):     # the staged copy is the library's packing of the same matrix
                assert np.array_equal(stack.host[l][e][0][m].numpy().reshape(p.shape), p)
                assert np.array_equal(stack.host[l][e][1][m].numpy().astype(np.float32).reshape(s_.shape), s_)
            return [p for p, _ in ps], [s_ for _, s_ in ps]

        def check(l, x, ids, gates, y, tokens, channels):
            worst, cache = 0.0, {}
            for t in tokens:
                acc = np.zeros(len(channels))
                for j in range(sh.top_k):
                    e = int(ids[t, j])
                    if e not in cache:
                        cache[e] = oracle_expert(l, e)
                    p, s_ = cache[e]
                    h = oracle.hidden_for_pair(x[t], sh.d_ff, sh.act, sh.group, True, bits[e], p, s_)
                    acc += float(gates[t, j]) * oracle.output_channels(h, sh.group, bits[e], p[2], s_[2], channels)
                worst = max(worst, float(np.abs(y[t, channels] - acc).max()))
            return worst / float(np.abs(y).max())

        channels = np.arange(3, sh.d_model, 131, dtype=np.int32)
        # prefill
        x_host = [inputs.activations(w.seed, l, T, sh.d_model, "bf16") for l in range(2)]
        xs = [torch.from_numpy(x).to(stack.dev).to(torch.bfloat16) for x in x_host]
        outs = []
        picks = stack.forward_stack(xs, outputs=outs)
        stack.compute.synchronize()
        assert B.emoe_device_status(stack.ctx, stack.compute.cuda_stream) == B.OK
        gates, y = outs[1][0].cpu().numpy(), outs[1][1].cpu().numpy()
        assert np.isfinite(y).all()
        e1 = int(picks[1][0, 0])
        owners = [t for t in range(T) if e1 in picks[1][t]]
        assert check(1, x_host[1], picks[1], gates, y, [owners[2], owners[-2]], channels) <= 2e-3
        # decode: three single-token steps, the last one checked on both layers
        for step in range(3):
            x_host = [inputs.activations(w.seed, l, 1, sh.d_model, "bf16", batch_tag=10 + step) for l in range(2)]
            xs = [torch.from_numpy(x).to(stack.dev).to(torch.bfloat16) for x in x_host]
            outs = []
            picks = stack.forward_stack(xs, outputs=outs)
        stack.compute.synchronize()
        assert B.emoe_device_status(stack.ctx, stack.compute.cuda_stream) == B.OK
        for l in range(2):
            gates, y = outs[l][0].cpu().numpy(), outs[l][1].cpu().numpy()
            assert check(l, x_host[l], picks[l], gates, y, [0], channels) <= 2e-3
        st = B.emoe_cache_get_stats(stack.ctx)
        assert st["bytes_copied"] > 0 and st["hits"] + st["misses"] > 0
    finally:
        stack.close()


def test_exposed_copy_time_is_counted_by_the_library_and_vanishes_when_everything_is_resident():
    """Section 3.3's pipeline invariants on the library's own counter: loading on demand leaves the
    compute stream waiting (exposed time > 0, and about the copy time of the bytes); once every
    expert sits in a slot the same acquires cost next to nothing; nothing is counted while the
    accounting is off."""
    shape = inputs.LayerShape(2048, 4096, 4, 2, "relu", "softmax_renorm", 128, "f16", "bf16")
    host = HostExperts(shape, 1, lambda l: [8, 8, 8, 8], seed=37)
    desc = layer.make_desc(shape)
    dev = torch.device("cuda", 0)
    torch.zeros(1, device=dev)
    ctx = B.emoe_create(0, B.emoe_workspace_bytes(desc, 4))
    compute, copy = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    model = ExpertBufferModel(4, 1, "forward")
    try:
        B.emoe_cache_create(ctx, 4, host.slot_bytes(), 1, B.EVICT_FORWARD)
        host.register_all(ctx, model)
        eids = [host.expert_id(0, e) for e in range(4)]
        B.emoe_cache_acquire(ctx, eids[:1], 0, compute.cuda_stream, copy.cuda_stream)     # accounting off
        B.emoe_cache_release(ctx, eids[:1], compute.cuda_stream)
        compute.synchronize()
        st = B.emoe_cache_get_stats(ctx)
        assert st["exposed_copy_ns"] == 0 and st["timed_acquires"] == 0
        B.emoe_cache_set_timing(ctx, True)
        B.emoe_cache_acquire(ctx, eids[1:], 0, compute.cuda_stream, copy.cuda_stream)     # three loads on demand
        B.emoe_cache_release(ctx, eids[1:], compute.cuda_stream)
        compute.synchronize()
        st1 = B.emoe_cache_get_stats(ctx)
        nbytes = sum(sum(host.nbytes(0, e)) for e in range(1, 4))                         # 3 x 16.9 MB
        assert st1["timed_acquires"] == 1
        assert st1["exposed_copy_ns"] > nbytes / 100e9 * 1e9          # no host link moves 100 GB/s
        assert st1["exposed_copy_ns"] < 1e9
        for _ in range(3):                                                                # everything resident now
            B.emoe_cache_acquire(ctx, eids, 0, compute.cuda_stream, copy.cuda_stream)
            B.emoe_cache_release(ctx, eids, compute.cuda_stream)
        compute.synchronize()
        st2 = B.emoe_cache_get_stats(ctx)
        assert st2["timed_acquires"] == 4 and st2["misses"] == st1["misses"]
        assert st2["exposed_copy_ns"] - st1["exposed_copy_ns"] < 0.05 * st1["exposed_copy_ns"]
    finally:
        torch.cuda.synchronize()
        B.emoe_destroy(ctx)


def test_tokens_per_expert_of_the_last_forward_call():
    shape = inputs.LayerShape(512, 1024, 8, 2, "relu", "softmax_renorm", 128, "f16", "bf16")
    bits = [8, 4, 2, 4, 8, 4, 2, 4]
    W = inputs.expert_set(39, 0, shape)
    Wr = inputs.router_weight(39, 0, shape.d_model, shape.n_experts, std=0.05)
    with layer.MoELayer(shape, bits, max_tokens=200) as moe:
        with pytest.raises(B.EmoeError):
            B.emoe_last_expert_counts(moe.ctx, shape.n_experts)      # no forward call yet
        moe.pack_from_host(W)
        for T in (1, 37, 200):                                        # streaming kernels and the grouped GEMM
            x = inputs.activations(39, T, T, shape.d_model, "bf16")
            _, ids, _, _ = moe.forward(x, Wr)
            counts = B.emoe_last_expert_counts(moe.ctx, shape.n_experts)
            assert np.array_equal(counts, np.bincount(ids.reshape(-1), minlength=shape.n_experts))
        with pytest.raises(B.EmoeError):
            B.emoe_last_expert_counts(moe.ctx, shape.n_experts + 1)
