"""Parity of the CUDA library (through the C ABI) with the CPU oracle, element by element, on the
same seeded inputs.  Integers (q_a, packed words, INT32 accumulators) must match bit for bit; fp32
outputs to max relative error 1e-5; bf16 outputs to 1 bf16 ulp."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift

pytestmark = pytest.mark.gpu

LEVELS = {"MNZ": (qift.MNZ, oracle.MNZ), "POT": (qift.POT, oracle.POT), "SYM": (qift.SYM, oracle.SYM),
          "INT4": (qift.INT4, oracle.INT4)}
assert all(a == b for a, b in LEVELS.values())


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def as_u32(t):
    return t.cpu().numpy().view(np.uint32).ravel()


def assert_status_clean():
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, f"device status {rc} detail {detail:#x}"


def check_outputs(y_gpu, acc_gpu, y_ref, acc_ref, bf16):
    assert np.array_equal(acc_gpu.cpu().numpy(), acc_ref), "INT32 accumulators differ"
    if bf16:
        got = y_gpu.view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int64)
        ref = y_ref.astype(np.int64)
        # ordered-integer distance between bf16 bit patterns = ulps
        key = lambda v: np.where(v & 0x8000, 0x8000 - (v & 0x7FFF), 0x8000 + v)
        assert np.abs(key(got) - key(ref)).max() <= 1
    else:
        got = y_gpu.cpu().numpy()
        denom = np.maximum(np.abs(y_ref), 1e-30)
        assert (np.abs(got - y_ref) / denom).max() <= 1e-5
        assert np.array_equal(got, y_ref)      # same two rounded multiplies in the same order


# ---------------------------------------------------------------------------------- rotation / K2
@pytest.mark.parametrize("M,K,B", [(1, 256, 256), (3, 4096, 4096), (5, 11008, 256), (4, 14336, 2048),
                                   (2, 512, 0), (7, 64, 4), (2, 16384, 16384), (33, 1024, 64), (1, 16, 2),
                                   (5, 4096, 1024), (3, 16384, 2048), (2, 2048, 1024), (9, 12288, 4096),  # 4, 8, 2, 3 blocks
                                   (3, 96, 32), (2, 224, 32), (4, 192, 64), (3, 640, 128), (2, 1536, 512), (3, 16384, 8192),
                                   (2, 8192, 8192), (2, 48, 16), (300, 4096, 4096), (150, 14336, 2048), (150, 11008, 256)])
@pytest.mark.parametrize("bf16", [False, True])
def test_quantize_act(M, K, B, bf16):
    x, _ = synth.activations(100 + M, M, K, max(1, K // 100))
    if bf16:
        xb = dev(x).to(torch.bfloat16)
        x_ref = oracle.bf16_to_f32(xb.view(torch.int16).cpu().numpy().view(np.uint16))
        q, s = qift.qift_quantize_act(xb, B, 0.9)
    else:
        x_ref = x
        q, s = qift.qift_quantize_act(dev(x), B, 0.9)
    q_ref, s_ref = oracle.quantize_act(x_ref, B, 0.9)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(s.cpu().numpy(), s_ref)
    assert_status_clean()


@pytest.mark.parametrize("M,K", [(3, 14336), (2, 448), (5, 7168)])
@pytest.mark.parametrize("bf16", [False, True])
def test_quantize_act_full_dimension_rotation(M, K, bf16):
    # K = 28 * 2^p with had_block = K: H_28 (x) H_{2^p}, bit-exact with the oracle (same summation order)
    x, _ = synth.activations(110 + M, M, K, max(1, K // 100))
    xd = dev(x)
    if bf16:
        xd = xd.to(torch.bfloat16)
        x = oracle.bf16_to_f32(xd.view(torch.int16).cpu().numpy().view(np.uint16))
    q, s = qift.qift_quantize_act(xd, K, 0.9)
    q_ref, s_ref = oracle.quantize_act(x, K, 0.9)
    assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)
    if not bf16:
        W = synth.student_weights(8, M, K)
        assert np.array_equal(qift.qift_rotate(dev(W), K).cpu().numpy(), oracle.rotate_weights(W, K))
    assert_status_clean()


def test_full_dimension_rotation_grouped_and_rejections():
    # a plan that mixes a full-dimension problem with a block-diagonal one
    lv, M = qift.MNZ, 2
    probs, refs = [], []
    for i, (N, K, B) in enumerate([(64, 14336, 14336), (48, 4096, 4096)]):
        W = synth.gaussian_weights(700 + i, N, K)
        x, _ = synth.activations(710 + i, M, K, 8)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
        refs.append(oracle.linear(codes, lv, s_n, q_ref, sa_ref))
        probs.append((dev(x), dev(p_ref.view(np.int32)), dev(s_n), B))
    plan = qift.qift_group_plan(probs, lv, 0.9, want_acc=True)
    outs = qift.qift_group_forward(plan)
    for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
        check_outputs(y, acc, y_ref, acc_ref, False)
    x = torch.zeros((1, 11008), device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_quantize_act(x, 11008, 0.9)                    # 11008 = 43 * 256: no construction for order 43 * 2^p here
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    assert_status_clean()


def test_quantize_act_zero_and_clip():
    x = np.zeros((2, 256), dtype=np.float32)
    x[1, 5] = -3.0
    for clip in (0.9, 1.0, 0.5):
        q, s = qift.qift_quantize_act(dev(x), 256, clip)
        q_ref, s_ref = oracle.quantize_act(x, 256, clip)
        assert np.array_equal(q.cpu().numpy(), q_ref) and np.array_equal(s.cpu().numpy(), s_ref)


@pytest.mark.parametrize("M,K,B", [(4, 256, 256), (3, 4096, 4096), (2, 11008, 256), (2, 14336, 2048), (5, 96, 32)])
def test_rotate(M, K, B):
    W = synth.student_weights(7, M, K)
    got = qift.qift_rotate(dev(W), B).cpu().numpy()
    assert np.array_equal(got, oracle.rotate_weights(W, B))
    w = dev(W)
    qift.qift_rotate(w, B, out=w)        # in place
    assert np.array_equal(w.cpu().numpy(), got)


# ---------------------------------------------------------------------------------- K1 packer
@pytest.mark.parametrize("name", list(LEVELS))
@pytest.mark.parametrize("N,K", [(256, 256), (37, 1024), (16, 11008), (3, 16), (50, 2320)])
def test_pack_absmax_and_given(name, N, K):
    lv = LEVELS[name][0]
    W = synth.gaussian_weights(0, N, K)
    W[N // 2] = 0                                   # a zero row
    W[0, :4] = [0.0, 1e-9, -1e-9, 0.0]
    packed, s_n = qift.qift_pack_weights(dev(W), lv, qift.SCALE_ABSMAX)
    p_ref, s_ref, codes_ref = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
    assert np.array_equal(s_n.cpu().numpy(), s_ref)
    assert np.array_equal(as_u32(packed), p_ref)
    # given scales, with weights sitting exactly on decision thresholds
    s_given = (np.abs(W).max(1) * 0.3 + 1e-3).astype(np.float32)
    Wt = W.copy()
    mids = np.array([-2.5, -2.0, -1.5, -0.5, 0.0, 0.5, 1.5, 2.0, 2.5, 7.5, -8.5], dtype=np.float32)
    if K >= len(mids):
        Wt[:, :len(mids)] = mids[None, :] * s_given[:, None]
    packed, s_out = qift.qift_pack_weights(dev(Wt), lv, qift.SCALE_GIVEN, s_n=dev(s_given))
    p_ref, _, _ = oracle.pack_weights(Wt, lv, oracle.SCALE_GIVEN, s_given)
    assert np.array_equal(as_u32(packed), p_ref)
    assert np.array_equal(s_out.cpu().numpy(), s_given)
    codes = qift.qift_unpack_codes(packed, N, K, lv).cpu().numpy()
    assert np.array_equal(codes, oracle.unpack(p_ref, N, K, lv))
    assert_status_clean()


@pytest.mark.parametrize("name", list(LEVELS))
def test_pack_mse(name):
    lv = LEVELS[name][0]
    N, K = 96, 4096
    W = oracle.rotate_weights(synth.student_weights(3, N, K), K)
    packed, s_n = qift.qift_pack_weights(dev(W), lv, qift.SCALE_MSE)
    s_gpu = s_n.cpu().numpy()
    s_ref, idx_ref, errs = oracle.weight_scale(W, lv, oracle.SCALE_MSE, want_errs=True)
    diff = np.nonzero(s_gpu != s_ref)[0]
    for n in diff:      # the sum order differs: only a numerical tie may change the winner
        e = np.sort(errs[n])
        assert (e[1] - e[0]) <= 1e-12 * e[0], f"row {n}: scale differs without a tie"
    # codes are exact given the scales the GPU chose
    p_ref, _, _ = oracle.pack_weights(W, lv, oracle.SCALE_GIVEN, s_gpu)
    assert np.array_equal(as_u32(packed), p_ref)
    assert len(diff) <= 1


# ---------------------------------------------------------------------------------- S4 + S5
def make_problem(lv, M, N, K, seed, B=None):
    W = synth.gaussian_weights(seed, N, K)
    x, _ = synth.activations(seed + 1, M, K, max(1, K // 100))
    if B is None:
        B = synth.had_block_for(K)
    p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
    q_a, s_a = oracle.quantize_act(x, B, 0.9)
    return p_ref, s_n, codes, q_a, s_a


def run_route(p_ref, s_n, lv, q_a, s_a, route, bf16):
    out_dtype = torch.bfloat16 if bf16 else torch.float32
    y, acc = qift.qift_linear_route(dev(p_ref.view(np.int32)), dev(s_n), lv, dev(q_a), dev(s_a), route,
                                    out_dtype=out_dtype, want_acc=True)
    assert_status_clean()
    return y, acc


@pytest.mark.parametrize("name", list(LEVELS))
@pytest.mark.parametrize("route", [qift.ROUTE_GENERIC, qift.ROUTE_DECODE, qift.ROUTE_DECODE_ROWS])
@pytest.mark.parametrize("M,N,K", [(1, 256, 256), (1, 40, 512), (3, 100, 2304), (8, 64, 4096), (9, 48, 1024),
                                   (16, 130, 2560), (5, 16, 11008), (2, 2400, 256), (2, 21, 48), (16, 4100, 512),
                                   (12, 300, 14336), (17, 200, 1024), (32, 1500, 512), (25, 140, 4096), (64, 300, 1024), (41, 130, 2560)])
def test_decode_routes(name, route, M, N, K):
    lv = LEVELS[name][0]
    if route != qift.ROUTE_GENERIC and K % 256:
        pytest.skip("the decode routes need whole 16-word slices")
    if route == qift.ROUTE_DECODE_ROWS and M == 1:
        pytest.skip("the row-split route starts at two token rows")
    if route == qift.ROUTE_DECODE and M > 16:
        pytest.skip("the K-split decode route ends at 16 token rows")
    p_ref, s_n, codes, q_a, s_a = make_problem(lv, M, N, K, seed=50 + M)
    for bf16 in (False, True):
        y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_a, s_a, bf16=bf16)
        y, acc = run_route(p_ref, s_n, lv, q_a, s_a, route, bf16)
        check_outputs(y, acc, y_ref, acc_ref, bf16)


@pytest.mark.parametrize("M", [1, 16, 40])
def test_linear_in_a_cuda_graph(M):
    # the per-call product captured once and replayed on new inputs: nothing in the launch may depend on host memory
    # that is gone at replay (the row-split route passes its one problem record by value)
    lv, N, K = qift.MNZ, 300, 1024
    p_ref, s_n, codes, q_a, s_a = make_problem(lv, M, N, K, seed=90)
    packed, sn, q, sa = dev(p_ref.view(np.int32)), dev(s_n), dev(q_a), dev(s_a)
    out = torch.empty((M, N), device="cuda")
    ws = torch.empty(max(256, qift.qift_workspace_bytes(M, N, K, lv)), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        qift.qift_w2a4_linear(packed, sn, lv, q, sa, out=out, workspace=ws)      # warm-up: attribute calls happen here
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            qift.qift_w2a4_linear(packed, sn, lv, q, sa, out=out, workspace=ws)
    for seed in (91, 92):
        _, _, _, q_new, sa_new = make_problem(lv, M, N, K, seed=seed)
        q.copy_(dev(q_new)), sa.copy_(dev(sa_new))
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        y_ref, _ = oracle.linear(codes, lv, s_n, q_new, sa_new)
        assert np.array_equal(out.cpu().numpy(), y_ref)
    assert_status_clean()


@pytest.mark.parametrize("name", ["MNZ", "INT4"])
def test_decode_extreme_values(name):
    # all codes at the top level against all activations at -8 / +7: the largest accumulators
    lv = LEVELS[name][0]
    N, K, M = 32, 14336, 2
    top = 15 if lv == qift.INT4 else 3
    codes = np.full((N, K), top if lv != qift.INT4 else 7, dtype=np.uint8)
    codes[1::2] = 0 if lv != qift.INT4 else 8                     # most negative level
    p_ref = oracle.pack(codes, lv)
    q_a = np.stack([np.full(K, 7, dtype=np.int8), np.full(K, -8, dtype=np.int8)])
    s_a = np.array([0.5, 2.0], dtype=np.float32)
    s_n = np.linspace(0.01, 0.02, N).astype(np.float32)
    y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_a, s_a)
    assert np.abs(acc_ref).max() == K * 8 * (8 if lv == qift.INT4 else 3)
    for route in (qift.ROUTE_GENERIC, qift.ROUTE_DECODE):
        y, acc = run_route(p_ref, s_n, lv, q_a, s_a, route, False)
        check_outputs(y, acc, y_ref, acc_ref, False)


@pytest.mark.parametrize("name", list(LEVELS))
@pytest.mark.parametrize("route", [qift.ROUTE_PREFILL, qift.ROUTE_PREFILL_SCRATCH, qift.ROUTE_PREFILL_PAIR,
                                   qift.ROUTE_PREFILL_FUSED_PAIR])
@pytest.mark.parametrize("M,N,K", [(128, 256, 512), (200, 300, 1024), (17, 72, 256), (512, 1024, 384), (130, 520, 4096),
                                   (300, 2000, 2320), (1, 40, 48)])
def test_prefill_route(name, route, M, N, K):
    lv = LEVELS[name][0]
    p_ref, s_n, codes, q_a, s_a = make_problem(lv, M, N, K, seed=80)
    for bf16 in (True, False):
        y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_a, s_a, bf16=bf16)
        y, acc = run_route(p_ref, s_n, lv, q_a, s_a, route, bf16)
        check_outputs(y, acc, y_ref, acc_ref, bf16)


def test_prefill_pair_route_224_wide_tiles():
    # 3 token-tile pairs x 3100 channels: one round of 224-wide tiles (42 of them) beats one round of
    # 256-wide and two rounds of 128-wide ones in the launcher's cost model, so this exercises the third
    # tile width, ragged in both directions (600 = 2*256 + 88 tokens, 3100 = 13*224 + 188 channels)
    lv = qift.MNZ
    p_ref, s_n, codes, q_a, s_a = make_problem(lv, 600, 3100, 256, seed=81)
    y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_a, s_a, bf16=True)
    for route in (qift.ROUTE_PREFILL_PAIR, qift.ROUTE_PREFILL_FUSED_PAIR):
        y, acc = run_route(p_ref, s_n, lv, q_a, s_a, route, True)
        check_outputs(y, acc, y_ref, acc_ref, True)
    assert_status_clean()


@pytest.mark.parametrize("name", list(LEVELS))
def test_resident_decoded_weights(name):
    # decode once to int8 levels, then the product alone: levels and outputs against the oracle
    lv = LEVELS[name][0]
    M, N, K = 300, 520, 1040
    p_ref, s_n, codes, q_a, s_a = make_problem(lv, M, N, K, seed=82)
    lev = qift.qift_expand_weights(dev(p_ref.view(np.int32)), N, K, lv)
    want = np.vectorize(lambda c: oracle.level_value(lv, int(c)))(codes).astype(np.int8)
    assert np.array_equal(lev.cpu().numpy(), want)
    for bf16 in (True, False):
        y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_a, s_a, bf16=bf16)
        y, acc = qift.qift_expanded_linear(lev, dev(s_n), dev(q_a), dev(s_a),
                                           out_dtype=torch.bfloat16 if bf16 else torch.float32, want_acc=True)
        check_outputs(y, acc, y_ref, acc_ref, bf16)
    assert_status_clean()


def test_auto_route_and_public_entry_points():
    for M in (1, 16, 17, 140):
        for lv in (qift.MNZ, qift.INT4):
            p_ref, s_n, codes, q_a, s_a = make_problem(lv, M, 96, 512, seed=9)
            y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_a, s_a)
            args = (dev(p_ref.view(np.int32)), dev(s_n))
            if lv == qift.INT4:
                y, acc = qift.qift_w4a4_linear(*args, dev(q_a), dev(s_a), want_acc=True)
            else:
                y, acc = qift.qift_w2a4_linear(*args, lv, dev(q_a), dev(s_a), want_acc=True)
            check_outputs(y, acc, y_ref, acc_ref, False)
    assert_status_clean()


def test_runs_are_deterministic():
    lv = qift.MNZ
    p_ref, s_n, codes, q_a, s_a = make_problem(lv, 4, 512, 4096, seed=4)
    outs = [run_route(p_ref, s_n, lv, q_a, s_a, qift.ROUTE_DECODE, False) for _ in range(3)]
    for y, acc in outs[1:]:
        assert torch.equal(y, outs[0][0]) and torch.equal(acc, outs[0][1])


# ---------------------------------------------------------------------------------- whole path
def test_whole_path_config1():
    # config 1: N = K = 256, M = 1, N(0, 0.02^2) weights (seed 0), 4 outlier channels x20, MNZ
    W = synth.gaussian_weights(0, 256, 256)
    x, _ = synth.activations(1, 1, 256, 4)
    for mode_g, mode_o in ((qift.SCALE_ABSMAX, oracle.SCALE_ABSMAX), (qift.SCALE_MSE, oracle.SCALE_MSE)):
        packed, s_n = qift.qift_pack_weights(dev(W), qift.MNZ, mode_g)
        q_a, s_a = qift.qift_quantize_act(dev(x), 256, 0.9)
        y, acc = qift.qift_w2a4_linear(packed, s_n, qift.MNZ, q_a, s_a, want_acc=True)
        p_ref, s_ref, codes = oracle.pack_weights(W, oracle.MNZ, mode_o)
        q_ref, sa_ref = oracle.quantize_act(x, 256, 0.9)
        y_ref, acc_ref = oracle.linear(codes, oracle.MNZ, s_ref, q_ref, sa_ref)
        assert np.array_equal(as_u32(packed), p_ref) and np.array_equal(s_n.cpu().numpy(), s_ref)
        assert np.array_equal(q_a.cpu().numpy(), q_ref) and np.array_equal(s_a.cpu().numpy(), sa_ref)
        check_outputs(y, acc, y_ref, acc_ref, False)
    assert_status_clean()


# ---------------------------------------------------------------------------------- whole layer in one call
@pytest.mark.parametrize("name", list(LEVELS))
@pytest.mark.parametrize("M,N,K,B", [(1, 300, 1024, 1024), (5, 130, 2560, 512), (16, 260, 4096, 4096), (40, 200, 1024, 0),
                                     (100, 96, 512, 256), (3, 64, 14336, 14336), (9, 40, 11008, 256)])
def test_forward_one_call(name, M, N, K, B):
    # rotation + activation quantization + product + scales in one call, on device tensors and through host buffers;
    # 2..64 rows go through the grouped path's quantizer and the row-split kernel, the rest through the per-call kernels
    lv = LEVELS[name][0]
    W = synth.gaussian_weights(900 + M, N, K)
    x, _ = synth.activations(901 + M, M, K, max(1, K // 100))
    p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
    packed, sn = dev(p_ref.view(np.int32)), dev(s_n)
    for bf16_in in (False, True):
        xd = dev(x).to(torch.bfloat16) if bf16_in else dev(x)
        x_ref = oracle.bf16_to_f32(xd.view(torch.int16).cpu().numpy().view(np.uint16)) if bf16_in else x
        q_ref, sa_ref = oracle.quantize_act(x_ref, B, 0.9)
        for bf16_out in (False, True):
            y_ref, _ = oracle.linear(codes, lv, s_n, q_ref, sa_ref, bf16=bf16_out)
            y = qift.qift_forward(xd, B, packed, sn, lv, out_dtype=torch.bfloat16 if bf16_out else torch.float32)
            assert_status_clean()
            if bf16_out:
                got = y.view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int64)
                key = lambda v: np.where(v & 0x8000, 0x8000 - (v & 0x7FFF), 0x8000 + v)
                assert np.abs(key(got) - key(y_ref.astype(np.int64))).max() <= 1
            else:
                assert np.array_equal(y.cpu().numpy(), y_ref)
    # host buffers in and out
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty((M, N), dtype=torch.float32).pin_memory()
    qift.qift_forward_host(xh, B, packed, sn, lv, yh)
    torch.cuda.synchronize()
    q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
    y_ref, _ = oracle.linear(codes, lv, s_n, q_ref, sa_ref)
    assert np.array_equal(yh.numpy(), y_ref)
    assert_status_clean()


# ---------------------------------------------------------------------------------- grouped path
@pytest.mark.parametrize("name", list(LEVELS))
@pytest.mark.parametrize("M", [1, 2, 5, 6, 8, 9, 13, 16, 17, 27, 32, 33, 50, 64, 65, 100, 128])
def test_grouped_forward(name, M):
    # a ragged list: different N (incl. not a multiple of the row block), different K (incl. a
    # partial last chunk), more items than CTAs
    lv = LEVELS[name][0]
    shapes = [(256, 256), (40, 512), (100, 2304), (4000, 256), (48, 4096), (130, 2560), (16, 11008), (2400, 256),
              (9600, 256)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        W = synth.gaussian_weights(300 + i, N, K)
        x, _ = synth.activations(400 + i, M, K, max(1, K // 100))
        B = synth.had_block_for(K)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
        y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_ref, sa_ref)
        probs.append((dev(x), dev(p_ref.view(np.int32)), dev(s_n), B))
        refs.append((q_ref, sa_ref, y_ref, acc_ref))
    plan = qift.qift_group_plan(probs, lv, 0.9, want_acc=True)
    for _ in range(2):      # a plan is reusable
        outs = qift.qift_group_forward(plan)
        assert_status_clean()
        for (q_ref, sa_ref, y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
            check_outputs(y, acc, y_ref, acc_ref, False)
    # the two halves separately
    qift.qift_group_quantize_act(plan)
    qift.qift_group_linear(plan)
    assert_status_clean()
    check_outputs(plan.outputs[2], plan.accs[2], refs[2][2], refs[2][3], False)


@pytest.mark.parametrize("name", list(LEVELS))
@pytest.mark.parametrize("M", [9, 16])
def test_grouped_forward_long_list(name, M):
    # a list long enough (>= two 256-row items per SM) for the plan to give every warp two row tiles; ragged N:
    # a last item with a single valid tile, one with a half-filled second tile of a warp, short last chunks of K
    lv = LEVELS[name][0]
    shapes = [(8200, 256), (8192, 512), (8472, 256), (8192, 256), (8000, 384 if lv == oracle.INT4 else 768), (8192, 256),
              (8192, 256), (8192, 256), (8192, 256), (8192, 256)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        W = synth.gaussian_weights(800 + i, N, K)
        x, _ = synth.activations(820 + i, M, K, max(1, K // 100))
        B = synth.had_block_for(K)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
        refs.append(oracle.linear(codes, lv, s_n, q_ref, sa_ref))
        probs.append((dev(x), dev(p_ref.view(np.int32)), dev(s_n), B))
    plan = qift.qift_group_plan(probs, lv, 0.9, want_acc=True)
    outs = qift.qift_group_forward(plan)
    assert_status_clean()
    for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
        check_outputs(y, acc, y_ref, acc_ref, False)


@pytest.mark.parametrize("name", ["MNZ", "SYM", "INT4", "POT"])
@pytest.mark.parametrize("M", [33, 64, 96, 128])
def test_grouped_forward_tensor_memory_kernel_many_items(name, M):
    # 33 .. 128 token rows of a plan run on the tcgen05 kernel whose weight operand lives in tensor memory.  More
    # 256-channel items than SMs, so CTAs take several items each (both accumulator buffers, the operand ring wrapping
    # across item boundaries); an odd number of 16-word slices per item (the two expander warps of a lane quarter swap
    # parity from item to item); ragged N: a last item with one valid 128-channel block, rows beyond N inside a block
    lv = LEVELS[name][0]
    k_odd = 1408 if lv == oracle.INT4 else 2816          # 11 slices per item
    shapes = [(33000, 512), (2304, 4096), (1000, k_odd), (6200, 1024), (300, 256)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        rng = np.random.default_rng(900 + i)
        codes = rng.integers(0, 16 if lv == oracle.INT4 else 4, (N, K), dtype=np.uint8)
        s_n = (0.005 + 0.01 * rng.random(N)).astype(np.float32)
        x, _ = synth.activations(920 + i, M, K, max(1, K // 100))
        B = synth.had_block_for(K)
        q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
        refs.append(oracle.linear(codes, lv, s_n, q_ref, sa_ref))
        probs.append((dev(x), dev(oracle.pack(codes, lv).view(np.int32)), dev(s_n), B))
    plan = qift.qift_group_plan(probs, lv, 0.9, want_acc=True)
    for _ in range(2):          # twice: the second run starts from the first one's tensor-memory and shared-memory contents
        outs = qift.qift_group_forward(plan)
        assert_status_clean()
        for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
            check_outputs(y, acc, y_ref, acc_ref, False)


@pytest.mark.parametrize("M", [1, 7])
def test_grouped_shared_activation(M):
    # q/k/v-style and gate/up-style modules read one activation: the plan quantizes it once (the buffers of the
    # sharing problems are the same) and every product still matches the oracle
    lv = oracle.MNZ
    K = 1024
    x1, _ = synth.activations(700, M, K, 8)
    x2, _ = synth.activations(701, M, K, 8)
    X1, X2 = dev(x1), dev(x2)
    probs, refs = [], []
    for i, (X, x, N) in enumerate([(X1, x1, 256), (X1, x1, 64), (X2, x2, 512), (X1, x1, 96), (X2, x2, 48)]):
        W = synth.gaussian_weights(710 + i, N, K)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x, 256, 0.9)
        refs.append(oracle.linear(codes, lv, s_n, q_ref, sa_ref))
        probs.append((X, dev(p_ref.view(np.int32)), dev(s_n), 256))
    for share in (True, False):
        plan = qift.qift_group_plan(probs, lv, 0.9, want_acc=True, share=share)
        q_ptrs = {plan.keep[5 * i + 3].data_ptr() for i in range(5)}
        assert len(q_ptrs) == (2 if share else 5)
        outs = qift.qift_group_forward(plan)
        assert_status_clean()
        for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
            check_outputs(y, acc, y_ref, acc_ref, False)
    # same X with a different rotation does not share
    plan = qift.qift_group_plan([probs[0], (X1, probs[1][1], probs[1][2], 128)], lv, 0.9, want_acc=True)
    assert plan.keep[3].data_ptr() != plan.keep[8].data_ptr()
    qift.qift_group_forward(plan)
    q128, sa128 = oracle.quantize_act(x1, 128, 0.9)
    W = synth.gaussian_weights(711, 64, K)
    _, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
    y_ref, acc_ref = oracle.linear(codes, lv, s_n, q128, sa128)
    check_outputs(plan.outputs[1], plan.accs[1], y_ref, acc_ref, False)


@pytest.mark.parametrize("M", [1, 12])
def test_grouped_forward_in_a_cuda_graph(M):
    # a plan captured once and replayed after the activations changed in place
    lv = qift.POT
    probs, packs = [], []
    for i, (N, K) in enumerate([(300, 1024), (64, 2560), (4100, 512)]):
        W = synth.gaussian_weights(950 + i, N, K)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        x, _ = synth.activations(960 + i, M, K, 8)
        probs.append((dev(x), dev(p_ref.view(np.int32)), dev(s_n), synth.had_block_for(K)))
        packs.append((codes, s_n, K))
    plan = qift.qift_group_plan(probs, lv, 0.9)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        qift.qift_group_forward(plan)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            qift.qift_group_forward(plan)
    for rnd in (1, 2):
        xs = []
        for i, (X, _, _, _) in enumerate(probs):
            x, _ = synth.activations(970 + 10 * rnd + i, M, X.shape[1], 8)
            X.copy_(dev(x))
            xs.append(x)
        g.replay()
        torch.cuda.synchronize()
        for (codes, s_n, K), x, y in zip(packs, xs, plan.outputs):
            q_ref, sa_ref = oracle.quantize_act(x, synth.had_block_for(K), 0.9)
            y_ref, _ = oracle.linear(codes, lv, s_n, q_ref, sa_ref)
            assert np.array_equal(y.cpu().numpy(), y_ref)
    assert_status_clean()


def test_grouped_rejects_bad_plans():
    x = torch.zeros((1, 256), device="cuda")
    packed = torch.zeros((16, 16), dtype=torch.int32, device="cuda")
    s_n = torch.ones(16, device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_group_plan([(x, packed, s_n, 96)], qift.MNZ)          # had_block not a power of two
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    x129 = torch.zeros((129, 256), device="cuda")
    with pytest.raises(qift.QiftError) as e:
        qift.qift_group_plan([(x129, packed, s_n, 256)], qift.MNZ)      # M > 128
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    L = qift.lib()
    assert L.qift_group_forward(None, None, None) == qift.ERR_INVALID_ARG


def test_grouped_forward_host_arenas():
    lv = qift.MNZ
    probs, refs = [], []
    for i, (N, K) in enumerate([(256, 256), (96, 512), (40, 1024)]):
        W = synth.gaussian_weights(500 + i, N, K)
        x, _ = synth.activations(600 + i, 2, K, 3)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x, synth.had_block_for(K), 0.9)
        refs.append(oracle.linear(codes, lv, s_n, q_ref, sa_ref)[0])
        probs.append((dev(x), dev(p_ref.view(np.int32)), dev(s_n), synth.had_block_for(K)))
    plan = qift.qift_group_plan(probs, lv, 0.9, arenas=True)
    plan.x_arena.zero_()                       # the device copy must come from the host arena
    y_host = qift.qift_group_forward_host(plan)
    torch.cuda.synchronize()
    assert_status_clean()
    for ref, y in zip(refs, plan.outputs):
        assert np.array_equal(y.cpu().numpy(), ref)
    off = 0
    for ref in refs:                           # and the host arena holds the same bytes
        n = ref.size * 4
        got = y_host[off:off + n].view(torch.float32).numpy().reshape(ref.shape)
        assert np.array_equal(got, ref)
        off += (n + 255) // 256 * 256
