"""The five benchmark configurations at (or close to) full size, CUDA path against the oracle.

Where the oracle would need minutes (the MSE sweep over a 45 M-weight matrix, a 2048-token product)
the comparison follows the sampled procedure: the GPU's scales are checked on a row sample, codes are
checked exactly for the whole matrix given those scales, and M = 2048 outputs are checked on sampled
token rows (all channels) and sampled channels (all tokens)."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift

pytestmark = pytest.mark.gpu
CLIP = 0.9


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def clean():
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, (rc, detail)


def rotated_t_weights(seed, N, K):
    """0.02 * t5 weights rotated along K by the blockwise Hadamard (the oracle's S0)."""
    return oracle.rotate_weights(synth.student_weights(seed, N, K), synth.had_block_for(K))


def pack_and_check(W, lv, mode, sample_rows=48):
    """GPU pack; scales checked against the oracle on a row sample, codes exactly for every row."""
    N, K = W.shape
    packed, s_n = qift.qift_pack_weights(dev(W), lv, mode)
    s_gpu = s_n.cpu().numpy()
    rows = np.linspace(0, N - 1, min(sample_rows, N)).astype(int)
    omode = {qift.SCALE_ABSMAX: oracle.SCALE_ABSMAX, qift.SCALE_MSE: oracle.SCALE_MSE}[mode]
    s_ref, _, errs = oracle.weight_scale(W[rows], lv, omode, want_errs=True)
    for j in np.nonzero(s_gpu[rows] != s_ref)[0]:
        e = np.sort(errs[j])
        assert omode == oracle.SCALE_MSE and (e[1] - e[0]) <= 1e-12 * e[0], f"row {rows[j]}: scale differs without a tie"
    codes = oracle.assign_codes(W, lv, s_gpu)
    assert np.array_equal(packed.cpu().numpy().view(np.uint32).ravel(), oracle.pack(codes, lv))
    return packed, s_n, codes, s_gpu


def check_module(packed, s_n, codes, s_gpu, lv, x, M, bf16_out=False, route=qift.ROUTE_AUTO):
    K = x.shape[1]
    B = synth.had_block_for(K)
    q_a, s_a = qift.qift_quantize_act(dev(x), B, CLIP)
    q_ref, sa_ref = oracle.quantize_act(x, B, CLIP)
    assert np.array_equal(q_a.cpu().numpy(), q_ref) and np.array_equal(s_a.cpu().numpy(), sa_ref)
    y, acc = qift.qift_linear_route(packed, s_n, lv, q_a, s_a, route, want_acc=True,
                                    out_dtype=torch.bfloat16 if bf16_out else torch.float32)
    y_ref, acc_ref = oracle.linear(codes, lv, s_gpu, q_ref, sa_ref, bf16=bf16_out)
    assert np.array_equal(acc.cpu().numpy(), acc_ref)
    got = y.view(torch.int16).cpu().numpy().view(np.uint16) if bf16_out else y.cpu().numpy()
    assert np.array_equal(got, y_ref)


# ---------------------------------------------------------------------------------------- config 2
@pytest.mark.parametrize("shape_idx", [0, 4, 6])          # q (= k, v, o), gate (= up), down
def test_config2_llama2_decode_m1(shape_idx):
    name, N, K = synth.LLAMA2_7B[shape_idx]
    W = rotated_t_weights(synth.config_seed(2, shape_idx, 0), N, K)
    packed, s_n, codes, s_gpu = pack_and_check(W, qift.MNZ, qift.SCALE_MSE)
    x, _ = synth.activations(synth.config_seed(2, shape_idx, 1), 1, K, round(0.01 * K))
    check_module(packed, s_n, codes, s_gpu, qift.MNZ, x, 1)
    clean()


def test_config2_grouped_layer():
    # the seven modules of a layer through the grouped API (one plan, two launches)
    mods = []
    for i, (name, N, K) in enumerate(synth.LLAMA2_7B):
        W = synth.gaussian_weights(synth.config_seed(2, i, 0), N, K)
        x, _ = synth.activations(synth.config_seed(2, i, 1), 1, K, round(0.01 * K))
        p_ref, s_n, codes = oracle.pack_weights(W, oracle.MNZ, oracle.SCALE_ABSMAX)
        mods.append((x, p_ref, s_n, codes, synth.had_block_for(K)))
    plan = qift.qift_group_plan([(dev(x), dev(p.view(np.int32)), dev(s), B) for x, p, s, c, B in mods], qift.MNZ, CLIP,
                                want_acc=True)
    outs = qift.qift_group_forward(plan)
    clean()
    for (x, p, s_n, codes, B), y, acc in zip(mods, outs, plan.accs):
        q_ref, sa_ref = oracle.quantize_act(x, B, CLIP)
        y_ref, acc_ref = oracle.linear(codes, oracle.MNZ, s_n, q_ref, sa_ref)
        assert np.array_equal(acc.cpu().numpy(), acc_ref) and np.array_equal(y.cpu().numpy(), y_ref)


# ---------------------------------------------------------------------------------------- config 3
@pytest.mark.parametrize("shape_idx", [0, 1, 4, 6])       # q/o, k/v, gate/up, down
def test_config3_llama31_batched_decode(shape_idx):
    name, N, K = synth.LLAMA31_8B[shape_idx]
    W = rotated_t_weights(synth.config_seed(3, shape_idx, 0), N, K)
    for lv in (qift.POT, qift.SYM):
        packed, s_n, codes, s_gpu = pack_and_check(W, lv, qift.SCALE_ABSMAX)
        for M in (1, 4, 16):
            x, _ = synth.activations(synth.config_seed(3, shape_idx, 1) + M, M, K, round(0.01 * K))
            check_module(packed, s_n, codes, s_gpu, lv, x, M)
    clean()


@pytest.mark.parametrize("M", [64, 128])
def test_config3_shapes_grouped_plan_mid_m_bf16(M):
    # the launch configuration of the benchmark's mid_m block: LLaMA-3.1-8B shapes in one grouped plan, bf16 in and
    # out, 64 / 128 token rows (the tcgen05 weight-streaming kernel); q/o, k/v shapes whole, gate/up and down cut to
    # 1024 channels so that the oracle stays in seconds
    shapes = [(4096, 4096), (1024, 4096), (1024, 4096), (1024, 14336)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        W = synth.gaussian_weights(synth.config_seed(3, i, 0) + 7, N, K)
        x, _ = synth.activations(synth.config_seed(3, i, 1) + 7, M, K, round(0.01 * K))
        xd = dev(x).to(torch.bfloat16)
        x_ref = oracle.bf16_to_f32(xd.view(torch.int16).cpu().numpy().view(np.uint16))
        B = synth.had_block_for(K)
        p_ref, s_n, codes = oracle.pack_weights(W, oracle.MNZ, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x_ref, B, CLIP)
        refs.append(oracle.linear(codes, oracle.MNZ, s_n, q_ref, sa_ref, bf16=True))
        probs.append((xd, dev(p_ref.view(np.int32)), dev(s_n), B))
    plan = qift.qift_group_plan(probs, qift.MNZ, CLIP, out_dtype=torch.bfloat16, want_acc=True)
    outs = qift.qift_group_forward(plan)
    clean()
    for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
        assert np.array_equal(y.view(torch.int16).cpu().numpy().view(np.uint16), y_ref)


# ---------------------------------------------------------------------------------------- config 4
@pytest.mark.parametrize("shape_idx", [0, 1, 4, 6])
def test_config4_prefill_m2048_sampled(shape_idx):
    name, N, K = synth.LLAMA31_8B[shape_idx]
    M = 2048
    W = synth.gaussian_weights(synth.config_seed(4, shape_idx, 0), N, K)
    packed, s_n, codes, s_gpu = pack_and_check(W, qift.MNZ, qift.SCALE_ABSMAX)
    x, _ = synth.activations(synth.config_seed(4, shape_idx, 1), M, K, round(0.01 * K))
    xb = dev(x).to(torch.bfloat16)
    x_ref = oracle.bf16_to_f32(xb.view(torch.int16).cpu().numpy().view(np.uint16))
    B = synth.had_block_for(K)
    q_a, s_a = qift.qift_quantize_act(xb, B, CLIP)
    q_ref, sa_ref = oracle.quantize_act(x_ref, B, CLIP)
    assert np.array_equal(q_a.cpu().numpy(), q_ref) and np.array_equal(s_a.cpu().numpy(), sa_ref)
    y, acc = qift.qift_w2a4_linear(packed, s_n, qift.MNZ, q_a, s_a, out_dtype=torch.bfloat16, want_acc=True)
    clean()
    yb = y.view(torch.int16).cpu().numpy().view(np.uint16)
    acc = acc.cpu().numpy()
    rng = np.random.default_rng(shape_idx)
    rows = np.sort(rng.choice(M, 16, replace=False))        # sampled token rows, every channel
    y_ref, acc_ref = oracle.linear(codes, oracle.MNZ, s_gpu, q_ref[rows], sa_ref[rows], bf16=True)
    assert np.array_equal(acc[rows], acc_ref) and np.array_equal(yb[rows], y_ref)
    cols = np.sort(rng.choice(N, 64, replace=False))        # sampled channels, every token
    y_ref, acc_ref = oracle.linear(codes[cols], oracle.MNZ, s_gpu[cols], q_ref, sa_ref, bf16=True)
    assert np.array_equal(acc[:, cols], acc_ref) and np.array_equal(yb[:, cols], y_ref)
    # properties that hold at any size
    assert np.abs(acc).max() <= K * 3 * 8


# ---------------------------------------------------------------------------------------- config 5
def run_mixed_stack(shapes, n_layers, n_w4, M, check_every_module=True):
    """Layer-wise mixed precision: layers [0, n_w4) INT4, the rest MNZ; the chaining glue of the
    linear stack in fp32 (h -> q,k,v; a := v; o; h2 = h + o; g,u; d = relu(g) * u; h' = h2 + down d,
    then a per-token rescale to unit max).
    Every module is checked against the oracle on the GPU's actual input (teacher forcing)."""
    K_h = shapes[0][2]
    h = dev(synth.activations(5001, M, K_h, max(1, round(0.01 * K_h)))[0])
    checks = 0
    for layer in range(n_layers):
        lv = qift.INT4 if layer < n_w4 else qift.MNZ
        mods = {}
        for i, (name, N, K) in enumerate(shapes):
            W = synth.gaussian_weights(synth.config_seed(5, i, 0) + 100 * layer, N, K)
            p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
            mods[name] = (dev(p_ref.view(np.int32)), dev(s_n), codes, s_n, N, K)

        def module(name, x_gpu):
            nonlocal checks
            packed, s_n_d, codes, s_n, N, K = mods[name]
            B = synth.had_block_for(K)
            q_a, s_a = qift.qift_quantize_act(x_gpu, B, CLIP)
            if lv == qift.INT4:
                y, acc = qift.qift_w4a4_linear(packed, s_n_d, q_a, s_a, want_acc=True)
            else:
                y, acc = qift.qift_w2a4_linear(packed, s_n_d, lv, q_a, s_a, want_acc=True)
            if check_every_module:
                x_np = x_gpu.cpu().numpy()
                q_ref, sa_ref = oracle.quantize_act(x_np, B, CLIP)
                y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_ref, sa_ref)
                assert np.array_equal(q_a.cpu().numpy(), q_ref) and np.array_equal(s_a.cpu().numpy(), sa_ref)
                assert np.array_equal(acc.cpu().numpy(), acc_ref) and np.array_equal(y.cpu().numpy(), y_ref)
                checks += 1
            return y

        q, k, v = module("q", h), module("k", h), module("v", h)
        a = v if v.shape[1] == K_h else v.repeat(1, K_h // v.shape[1])   # grouped-query shapes: tile v up
        o = module("o", a)
        h2 = h + o
        g, u = module("gate", h2), module("up", h2)
        d_in = torch.clamp_min(g, 0.0) * u
        h = h2 + module("down", d_in)
        # there is no normalisation layer in this linear-only stack: rescale each token so that 32
        # layers of gated products stay finite (inputs must be finite; the glue is not under test)
        h = h / h.abs().amax(dim=1, keepdim=True).clamp_min(1e-30)
        assert torch.isfinite(h).all()
    clean()
    return checks


def test_config5_mixed_stack_full_shapes_two_layers():
    # one W4A4 layer followed by one W2A4 layer at the real LLaMA-2-7B shapes, M = 1
    assert run_mixed_stack(synth.LLAMA2_7B, 2, 1, 1) == 14


def test_config5_mixed_stack_32_layers_scaled_shapes():
    # the whole L = 16 layout (layers 0-15 INT4, 16-31 MNZ) on proportionally reduced shapes
    # (ffn width 768 = 3 * 256 keeps K a multiple of 256, as every LLaMA K is)
    small = [("q", 256, 256), ("k", 256, 256), ("v", 256, 256), ("o", 256, 256),
             ("gate", 768, 256), ("up", 768, 256), ("down", 256, 768)]
    assert run_mixed_stack(small, 32, 16, 1) == 224
    assert run_mixed_stack(small, 4, 2, 40) == 28           # the same stack through the prefill route


# ------------------------------------------------------------------- config 5 at M = 2048, full shapes
def prefill_module_sampled(pool, W, lv, x_bf16, seed, rows_n=64, cols_n=256):
    """One module at M = 2048 through the AUTO route (code expansion into the int8 scratch, then the CTA-pair
    tcgen05 GEMM), bf16 in and out.  INT32 accumulators and bf16 bits are compared with the oracle on `rows_n`
    seeded token rows x every channel and on every token x `cols_n` seeded channels.  The oracle jobs go to
    `pool` (the oracle itself stays single-threaded; independent calls run side by side) and are returned as
    thunks that do the comparison."""
    N, K = W.shape
    M = x_bf16.shape[0]
    B = synth.had_block_for(K)
    p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
    packed, s_d = dev(p_ref.view(np.int32)), dev(s_n)
    x_ref = oracle.bf16_to_f32(x_bf16.view(torch.int16).cpu().numpy().view(np.uint16))
    q_a, s_a = qift.qift_quantize_act(x_bf16, B, CLIP)
    q_ref, sa_ref = oracle.quantize_act(x_ref, B, CLIP)
    assert np.array_equal(q_a.cpu().numpy(), q_ref) and np.array_equal(s_a.cpu().numpy(), sa_ref)
    if lv == qift.INT4:
        y, acc = qift.qift_w4a4_linear(packed, s_d, q_a, s_a, out_dtype=torch.bfloat16, want_acc=True)
    else:
        y, acc = qift.qift_w2a4_linear(packed, s_d, lv, q_a, s_a, out_dtype=torch.bfloat16, want_acc=True)
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(M, rows_n, replace=False))
    cols = np.sort(rng.choice(N, cols_n, replace=False))
    rows_t, cols_t = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
    yb = y.view(torch.int16)
    got = (acc[rows_t].cpu().numpy(), yb[rows_t].cpu().numpy().view(np.uint16),
           acc[:, cols_t].cpu().numpy(), yb[:, cols_t].cpu().numpy().view(np.uint16))
    assert int(acc.abs().max()) <= K * 8 * 8           # holds at any size: |level| <= 8, |q_a| <= 8
    job_r = pool.submit(oracle.linear, codes, lv, s_n, q_ref[rows], sa_ref[rows], True)
    job_c = pool.submit(oracle.linear, np.ascontiguousarray(codes[cols]), lv, s_n[cols], q_ref, sa_ref, True)

    def finish():
        y_r, acc_r = job_r.result()
        y_c, acc_c = job_c.result()
        assert np.array_equal(got[0], acc_r) and np.array_equal(got[1], y_r)
        assert np.array_equal(got[2], acc_c) and np.array_equal(got[3], y_c)
    return finish


@pytest.mark.parametrize("lv", [qift.INT4, qift.MNZ], ids=["w4a4_layer", "w2a4_layer"])
def test_config5_prefill_m2048_full_shapes_sampled(lv):
    # one layer of the mixed stack at the LLaMA-2-7B shapes and M = 2048: all seven modules, each on its own input
    from concurrent.futures import ThreadPoolExecutor
    M = 2048
    with ThreadPoolExecutor(max_workers=8) as pool:
        pending = []
        for i, (name, N, K) in enumerate(synth.LLAMA2_7B):
            W = synth.gaussian_weights(synth.config_seed(5, i, 0) + 7000 + lv, N, K)
            x, _ = synth.activations(synth.config_seed(5, i, 1) + 7000, M, K, round(0.01 * K))
            pending.append(prefill_module_sampled(pool, W, lv, dev(x).to(torch.bfloat16), 50 + i))
        clean()
        for finish in pending:
            finish()


@pytest.mark.parametrize("lv", [qift.POT, qift.SYM], ids=["pot", "sym"])
def test_prefill_m2048_gate_shape_other_level_sets(lv):
    # the remaining two-bit sets once at full size through the same route (11008 channels: 224-wide tiles, 43 of them)
    from concurrent.futures import ThreadPoolExecutor
    M, (name, N, K) = 2048, synth.LLAMA2_7B[4]
    W = synth.gaussian_weights(synth.config_seed(5, 4, 0) + 7100 + lv, N, K)
    x, _ = synth.activations(synth.config_seed(5, 4, 1) + 7100, M, K, round(0.01 * K))
    with ThreadPoolExecutor(max_workers=2) as pool:
        finish = prefill_module_sampled(pool, W, lv, dev(x).to(torch.bfloat16), 60 + lv)
        clean()
        finish()
