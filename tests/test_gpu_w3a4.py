"""W3A4 (three-bit weights, Eq. 1 with b = 3: the equal-budget point of Sec. 4.4) through the C ABI against the oracle.

Packed words (both planes), codes, INT32 accumulators and outputs are compared bit for bit: the packer in every scale
mode, every product route that serves the level set (generic, row-split decode from one token row, decode-to-int8
tensor-core GEMMs), the one-call forward, grouped plans, the multi-output forward with its decode-ahead chain, and the
largest accumulators the format can produce."""
import numpy as np
import pytest
import torch

import oracle
import synth
import paper_2606_02823_b200 as qift

pytestmark = pytest.mark.gpu
LV = qift.INT3
assert qift.INT3 == oracle.INT3


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def as_u32(t):
    return t.cpu().numpy().view(np.uint32).ravel()


def clean():
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, (rc, hex(detail))


def check(y, acc, y_ref, acc_ref, bf16=False):
    assert np.array_equal(acc.cpu().numpy(), acc_ref), "INT32 accumulators differ"
    got = y.view(torch.int16).cpu().numpy().view(np.uint16) if bf16 else y.cpu().numpy()
    assert np.array_equal(got, y_ref)


def make_problem(M, N, K, seed, B=None):
    W = synth.gaussian_weights(seed, N, K)
    x, _ = synth.activations(seed + 1, M, K, max(1, K // 100))
    if B is None:
        B = synth.had_block_for(K)
    p_ref, s_n, codes = oracle.pack_weights(W, LV, oracle.SCALE_ABSMAX)
    q_a, s_a = oracle.quantize_act(x, B, 0.9)
    return x, B, p_ref, s_n, codes, q_a, s_a


# ------------------------------------------------------------------------------------------ packer
@pytest.mark.parametrize("N,K", [(256, 256), (37, 1024), (16, 11008), (3, 32), (50, 2336), (130, 4096)])
def test_pack_absmax_given_and_unpack(N, K):
    W = synth.gaussian_weights(0, N, K)
    W[N // 2] = 0
    W[0, :4] = [0.0, 1e-9, -1e-9, 0.0]
    packed, s_n = qift.qift_pack_weights(dev(W), LV, qift.SCALE_ABSMAX)
    p_ref, s_ref, _ = oracle.pack_weights(W, LV, oracle.SCALE_ABSMAX)
    assert qift.qift_packed_bytes(N, K, LV) == p_ref.size * 4
    assert np.array_equal(s_n.cpu().numpy(), s_ref)
    assert np.array_equal(as_u32(packed), p_ref)
    # given scales, weights exactly on rounding ties and beyond the clip on both sides
    s_given = (np.abs(W).max(1) * 0.2 + 1e-3).astype(np.float32)
    Wt = W.copy()
    ties = np.array([-4.5, -3.5, -2.5, -1.5, -0.5, 0.0, 0.5, 1.5, 2.5, 3.5, 7.5, -8.5], dtype=np.float32)
    Wt[:, :len(ties)] = ties[None, :] * s_given[:, None]
    packed, s_out = qift.qift_pack_weights(dev(Wt), LV, qift.SCALE_GIVEN, s_n=dev(s_given))
    p_ref, _, codes_ref = oracle.pack_weights(Wt, LV, oracle.SCALE_GIVEN, s_given)
    assert np.array_equal(as_u32(packed), p_ref)
    assert np.array_equal(s_out.cpu().numpy(), s_given)
    codes = qift.qift_unpack_codes(packed, N, K, LV).cpu().numpy()
    assert np.array_equal(codes, codes_ref) and codes.max() <= 7
    clean()


def test_pack_mse():
    N, K = 96, 4096
    W = oracle.rotate_weights(synth.student_weights(3, N, K), K)
    packed, s_n = qift.qift_pack_weights(dev(W), LV, qift.SCALE_MSE)
    s_gpu = s_n.cpu().numpy()
    s_ref, _, errs = oracle.weight_scale(W, LV, oracle.SCALE_MSE, want_errs=True)
    diff = np.nonzero(s_gpu != s_ref)[0]
    for n in diff:      # the sum order differs: only a numerical tie may change the winner
        e = np.sort(errs[n])
        assert (e[1] - e[0]) <= 1e-12 * e[0], f"row {n}: scale differs without a tie"
    p_ref, _, _ = oracle.pack_weights(W, LV, oracle.SCALE_GIVEN, s_gpu)
    assert np.array_equal(as_u32(packed), p_ref)
    assert len(diff) <= 1
    clean()


def test_rejections():
    W = dev(synth.gaussian_weights(1, 16, 48))
    with pytest.raises(qift.QiftError) as e:       # K must be a whole number of high words
        qift.qift_pack_weights(W, LV, qift.SCALE_ABSMAX)
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    assert qift.qift_packed_bytes(16, 48, LV) == 0
    x, B, p_ref, s_n, codes, q_a, s_a = make_problem(4, 64, 256, 5)
    for route in (qift.ROUTE_DECODE, qift.ROUTE_PREFILL, qift.ROUTE_PREFILL_FUSED_PAIR):
        with pytest.raises(qift.QiftError) as e:
            qift.qift_linear_route(dev(p_ref.view(np.int32)), dev(s_n), LV, dev(q_a), dev(s_a), route)
        assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    xs = dev(synth.activations(9, 17, 256, 2)[0])
    with pytest.raises(qift.QiftError) as e:       # plans of this level set end at 16 token rows
        qift.qift_group_plan([(xs, dev(p_ref.view(np.int32)), dev(s_n), 256)], LV, 0.9)
    assert e.value.status == qift.ERR_UNSUPPORTED_SHAPE
    clean()


# ------------------------------------------------------------------------------------------ products
@pytest.mark.parametrize("route", [qift.ROUTE_GENERIC, qift.ROUTE_DECODE_ROWS])
@pytest.mark.parametrize("M,N,K", [(1, 256, 256), (1, 40, 512), (3, 100, 2304), (8, 64, 4096), (9, 48, 1024), (16, 130, 2560),
                                   (5, 16, 11008), (2, 2400, 256), (2, 21, 96), (16, 4100, 512), (12, 300, 14336), (1, 4096, 4096)])
def test_decode_routes(route, M, N, K):
    if route == qift.ROUTE_DECODE_ROWS and K % 256:
        pytest.skip("the row-split route needs whole 16-word slices")
    x, B, p_ref, s_n, codes, q_a, s_a = make_problem(M, N, K, seed=70 + M)
    for bf16 in (False, True):
        y_ref, acc_ref = oracle.linear(codes, LV, s_n, q_a, s_a, bf16=bf16)
        y, acc = qift.qift_linear_route(dev(p_ref.view(np.int32)), dev(s_n), LV, dev(q_a), dev(s_a), route,
                                        out_dtype=torch.bfloat16 if bf16 else torch.float32, want_acc=True)
        clean()
        check(y, acc, y_ref, acc_ref, bf16)


@pytest.mark.parametrize("route", [qift.ROUTE_PREFILL_SCRATCH, qift.ROUTE_PREFILL_PAIR])
@pytest.mark.parametrize("M,N,K", [(128, 256, 512), (200, 300, 1024), (17, 72, 256), (600, 520, 384), (130, 520, 4096), (300, 37, 96)])
def test_gemm_routes(route, M, N, K):
    x, B, p_ref, s_n, codes, q_a, s_a = make_problem(M, N, K, seed=90 + M)
    for bf16 in (False, True):
        y_ref, acc_ref = oracle.linear(codes, LV, s_n, q_a, s_a, bf16=bf16)
        y, acc = qift.qift_linear_route(dev(p_ref.view(np.int32)), dev(s_n), LV, dev(q_a), dev(s_a), route,
                                        out_dtype=torch.bfloat16 if bf16 else torch.float32, want_acc=True)
        clean()
        check(y, acc, y_ref, acc_ref, bf16)


def test_extreme_values():
    # every weight at the most negative level against activations at -8 and at +7; K = 14336: the largest accumulators
    N, K = 144, 14336
    for M in (1, 16, 40):
        for code, qv in ((4, -8), (4, 7), (3, 7), (7, -8)):
            codes = np.full((N, K), code, dtype=np.uint8)
            q_a = np.full((M, K), qv, dtype=np.int8)
            s_n = np.full(N, 0.01, dtype=np.float32)
            s_a = np.full(M, 0.5, dtype=np.float32)
            y_ref, acc_ref = oracle.linear(codes, LV, s_n, q_a, s_a)
            assert abs(int(acc_ref[0, 0])) == K * abs(oracle.level_value(LV, code)) * abs(qv)
            y, acc = qift.qift_w3a4_linear(dev(oracle.pack(codes, LV).view(np.int32)), dev(s_n), dev(q_a), dev(s_a), want_acc=True)
            check(y, acc, y_ref, acc_ref)
    clean()


def test_public_entry_point_picks_a_route_for_every_m():
    N, K = 272, 1024
    for M in (1, 7, 16, 17, 64, 300, 700):
        x, B, p_ref, s_n, codes, q_a, s_a = make_problem(M, N, K, seed=200 + M)
        y_ref, acc_ref = oracle.linear(codes, LV, s_n, q_a, s_a)
        y, acc = qift.qift_w3a4_linear(dev(p_ref.view(np.int32)), dev(s_n), dev(q_a), dev(s_a), want_acc=True)
        check(y, acc, y_ref, acc_ref)
        # without scratch the call still runs where the generic kernel can serve it
        if M <= 16:
            none = torch.empty(0, dtype=torch.uint8, device="cuda")
            y2 = qift.qift_w3a4_linear(dev(p_ref.view(np.int32)), dev(s_n), dev(q_a), dev(s_a), workspace=none)
            assert np.array_equal(y2.cpu().numpy(), y_ref)
    clean()


@pytest.mark.parametrize("M,N,K,B", [(1, 300, 1024, 1024), (5, 130, 2560, 512), (16, 260, 4096, 4096), (40, 200, 1024, 0),
                                     (3, 64, 14336, 14336), (9, 40, 11008, 256), (600, 264, 512, 512)])
def test_forward_one_call(M, N, K, B):
    W = synth.gaussian_weights(900 + M, N, K)
    x, _ = synth.activations(901 + M, M, K, max(1, K // 100))
    p_ref, s_n, codes = oracle.pack_weights(W, LV, oracle.SCALE_ABSMAX)
    packed, sn = dev(p_ref.view(np.int32)), dev(s_n)
    for bf16_in in (False, True):
        xd = dev(x).to(torch.bfloat16) if bf16_in else dev(x)
        x_ref = oracle.bf16_to_f32(xd.view(torch.int16).cpu().numpy().view(np.uint16)) if bf16_in else x
        q_ref, sa_ref = oracle.quantize_act(x_ref, B, 0.9)
        for bf16_out in (False, True):
            y_ref, _ = oracle.linear(codes, LV, s_n, q_ref, sa_ref, bf16=bf16_out)
            y = qift.qift_forward(xd, B, packed, sn, LV, out_dtype=torch.bfloat16 if bf16_out else torch.float32)
            clean()
            got = y.view(torch.int16).cpu().numpy().view(np.uint16) if bf16_out else y.cpu().numpy()
            assert np.array_equal(got, y_ref)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty((M, N), dtype=torch.float32).pin_memory()
    qift.qift_forward_host(xh, B, packed, sn, LV, yh)
    torch.cuda.synchronize()
    q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
    assert np.array_equal(yh.numpy(), oracle.linear(codes, LV, s_n, q_ref, sa_ref)[0])
    clean()


# ------------------------------------------------------------------------------------------ grouped plans
@pytest.mark.parametrize("M", [1, 2, 5, 8, 9, 13, 16])
def test_grouped_forward(M):
    # a ragged list: N not a multiple of the row block, a partial last chunk of K, more items than CTAs
    shapes = [(256, 256), (40, 512), (100, 2304), (4000, 256), (48, 4096), (130, 2560), (16, 11008), (2400, 256), (9600, 256)]
    probs, refs = [], []
    for i, (N, K) in enumerate(shapes):
        W = synth.gaussian_weights(300 + i, N, K)
        x, _ = synth.activations(400 + i, M, K, max(1, K // 100))
        B = synth.had_block_for(K)
        p_ref, s_n, codes = oracle.pack_weights(W, LV, oracle.SCALE_ABSMAX)
        q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
        refs.append(oracle.linear(codes, LV, s_n, q_ref, sa_ref))
        probs.append((dev(x), dev(p_ref.view(np.int32)), dev(s_n), B))
    plan = qift.qift_group_plan(probs, LV, 0.9, want_acc=True)
    for _ in range(2):
        outs = qift.qift_group_forward(plan)
        clean()
        for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
            check(y, acc, y_ref, acc_ref)


@pytest.mark.parametrize("M", [1, 16])
def test_grouped_llama_layer_shapes(M):
    # one LLaMA-2-7B layer at full size, packed on the GPU with swept scales; all outputs against the oracle
    probs, refs = [], []
    for i, (_, N, K) in enumerate(synth.LLAMA2_7B):
        W = synth.gaussian_weights(500 + i, N, K)
        x, _ = synth.activations(520 + i, M, K, max(1, K // 100))
        B = synth.had_block_for(K)
        packed, s_n = qift.qift_pack_weights(dev(W), LV, qift.SCALE_ABSMAX)
        p_ref, s_ref, codes = oracle.pack_weights(W, LV, oracle.SCALE_ABSMAX)
        assert np.array_equal(as_u32(packed), p_ref)
        q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
        refs.append(oracle.linear(codes, LV, s_ref, q_ref, sa_ref))
        probs.append((dev(x), packed, s_n, B))
    plan = qift.qift_group_plan(probs, LV, 0.9, want_acc=True)
    outs = qift.qift_group_forward(plan)
    clean()
    for (y_ref, acc_ref), y, acc in zip(refs, outs, plan.accs):
        check(y, acc, y_ref, acc_ref)


# ------------------------------------------------------------------------------------------ several outputs, decode-ahead
def make_weights(seed, Ns, K, lv):
    host, gpu = [], []
    for i, N in enumerate(Ns):
        W = synth.gaussian_weights(seed + i, N, K)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        host.append((codes, s_n))
        gpu.append((dev(p_ref.view(np.int32)), dev(s_n)))
    return host, gpu


def check_multi(host, lv, x, B, ys, accs):
    q_ref, sa_ref = oracle.quantize_act(x, B, 0.9)
    for (codes, s_n), y, acc in zip(host, ys, accs):
        y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_ref, sa_ref)
        check(y, acc, y_ref, acc_ref)


@pytest.mark.parametrize("M", [600, 40, 3])
def test_forward_multi_and_decode_ahead(M):
    # call 1 (two-bit codes) decodes call 2's three-bit codes ahead, call 2 those of call 3 (two-bit again)
    K1, K2, K3 = 512, 768, 256
    h1, g1 = make_weights(11, (520, 128), K1, qift.MNZ)
    h2, g2 = make_weights(21, (300, 136), K2, LV)
    h3, g3 = make_weights(31, (136, 264), K3, qift.SYM)
    x1, _ = synth.activations(41, M, K1, 5)
    x2, _ = synth.activations(42, M, K2, 7)
    x3, _ = synth.activations(43, M, K3, 3)
    cap = max(qift.qift_levels_bytes(K1, g1), qift.qift_levels_bytes(K2, g2), qift.qift_levels_bytes(K3, g3))
    bufs = [torch.full((cap,), 0x55, dtype=torch.uint8, device="cuda") for _ in range(2)]
    y1, a1 = qift.qift_forward_multi(dev(x1), 512, g1, qift.MNZ, 0.9, want_acc=True, levels_buf=bufs[0], levels_ready=False,
                                     ahead=(g2, K2, LV, bufs[1]))
    y2, a2 = qift.qift_forward_multi(dev(x2), 256, g2, LV, 0.9, want_acc=True, levels_buf=bufs[1], levels_ready=True,
                                     ahead=(g3, K3, qift.SYM, bufs[0]))
    y3, a3 = qift.qift_forward_multi(dev(x3), 256, g3, qift.SYM, 0.9, want_acc=True, levels_buf=bufs[0], levels_ready=True)
    check_multi(h1, qift.MNZ, x1, 512, y1, a1)
    check_multi(h2, LV, x2, 256, y2, a2)
    check_multi(h3, qift.SYM, x3, 256, y3, a3)
    # and without a chain: the call decodes its own codes
    y2, a2 = qift.qift_forward_multi(dev(x2), 256, g2, LV, 0.9, want_acc=True)
    check_multi(h2, LV, x2, 256, y2, a2)
    clean()


def test_resident_decoded_weights():
    M, N, K = 520, 300, 1024
    x, B, p_ref, s_n, codes, q_a, s_a = make_problem(M, N, K, seed=77)
    lv_i8 = qift.qift_expand_weights(dev(p_ref.view(np.int32)), N, K, LV)
    table = np.array(oracle.level_table(LV), dtype=np.int8)
    assert np.array_equal(lv_i8.cpu().numpy().reshape(N, K), table[codes])
    y, acc = qift.qift_expanded_linear(lv_i8, dev(s_n), dev(q_a), dev(s_a), want_acc=True)
    y_ref, acc_ref = oracle.linear(codes, LV, s_n, q_a, s_a)
    check(y, acc, y_ref, acc_ref)
    clean()
