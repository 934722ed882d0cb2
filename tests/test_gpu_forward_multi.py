"""qift_forward_multi: one rotated + quantized activation, several products, codes decoded ahead of their use.

Every output is compared with the oracle bit for bit (INT32 accumulators and outputs), on shapes that span several
channel tiles of every tile width with ragged tails, for every level set, with and without the decode-ahead chain
(call A decodes call B's codes during its own GEMM; call B then skips its decoding pass)."""
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


def make_weights(seed, Ns, K, lv):
    host, gpu = [], []
    for i, N in enumerate(Ns):
        W = synth.gaussian_weights(seed + i, N, K)
        p_ref, s_n, codes = oracle.pack_weights(W, lv, oracle.SCALE_ABSMAX)
        host.append((codes, s_n))
        gpu.append((dev(p_ref.view(np.int32)), dev(s_n)))
    return host, gpu


def check(host, lv, x, B, ys, accs, bf16):
    q_ref, sa_ref = oracle.quantize_act(x, B, CLIP)
    for (codes, s_n), y, acc in zip(host, ys, accs):
        y_ref, acc_ref = oracle.linear(codes, lv, s_n, q_ref, sa_ref, bf16=bf16)
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
        got = y.view(torch.int16).cpu().numpy().view(np.uint16) if bf16 else y.cpu().numpy()
        assert np.array_equal(got, y_ref)


def clean():
    rc, detail = qift.qift_device_status()
    assert rc == qift.OK, (rc, detail)


@pytest.mark.parametrize("lv", [qift.MNZ, qift.POT, qift.SYM, qift.INT4])
@pytest.mark.parametrize("M,Ns,K", [(600, (520, 136, 128), 512),        # pair GEMM: three segments, ragged widths
                                    (513, (1000,), 256),               # one segment, four 256-wide tiles, ragged M
                                    (40, (272, 64), 512),              # row-split decode route per output
                                    (1, (256, 256, 256, 144), 256),    # single token, four outputs
                                    (100, (200, 320), 256),            # fused prefill route per output
                                    (129, (200, 320), 256),            # the first token count of the pair GEMM: one half-empty tile
                                    (300, (200, 320), 256),            # two token tiles, the second ragged
                                    (1100, (520, 136), 256),           # five token tiles, ragged M
                                    (2100, (1000,), 256),              # nine token tiles
                                    (1024, (4800, 264), 128)])         # more channel tiles than CTA pairs
def test_forward_multi_matches_oracle(lv, M, Ns, K):
    host, gpu = make_weights(100 * lv + M, Ns, K, lv)
    x, _ = synth.activations(7 + M, M, K, max(1, K // 100))
    B = synth.had_block_for(K)
    for dt in (torch.float32, torch.bfloat16):
        ys, accs = qift.qift_forward_multi(dev(x), B, gpu, lv, CLIP, out_dtype=dt, want_acc=True)
        check(host, lv, x, B, ys, accs, dt == torch.bfloat16)
    clean()


@pytest.mark.parametrize("M", [700, 64])
def test_decode_ahead_chain(M):
    # three calls in a row; each decodes the next one's codes (another K, another level set) while it runs
    K1, K2, K3 = 512, 768, 256
    h1, g1 = make_weights(11, (520, 128), K1, qift.MNZ)
    h2, g2 = make_weights(21, (300,), K2, qift.INT4)
    h3, g3 = make_weights(31, (136, 136, 264), K3, qift.POT)
    x1, _ = synth.activations(41, M, K1, 5)
    x2, _ = synth.activations(42, M, K2, 7)
    x3, _ = synth.activations(43, M, K3, 3)
    cap = max(qift.qift_levels_bytes(K1, g1), qift.qift_levels_bytes(K2, g2), qift.qift_levels_bytes(K3, g3))
    bufs = [torch.full((cap,), 0x55, dtype=torch.uint8, device="cuda") for _ in range(2)]   # stale bytes to begin with
    for rounds in range(2):     # the second round starts from buffers that hold the first round's levels
        y1, a1 = qift.qift_forward_multi(dev(x1), synth.had_block_for(K1), g1, qift.MNZ, CLIP, want_acc=True, levels_buf=bufs[0],
                                         levels_ready=False, ahead=(g2, K2, qift.INT4, bufs[1]))
        y2, a2 = qift.qift_forward_multi(dev(x2), synth.had_block_for(K2), g2, qift.INT4, CLIP, want_acc=True, levels_buf=bufs[1],
                                         levels_ready=True, ahead=(g3, K3, qift.POT, bufs[0]))
        y3, a3 = qift.qift_forward_multi(dev(x3), synth.had_block_for(K3), g3, qift.POT, CLIP, want_acc=True, levels_buf=bufs[0],
                                         levels_ready=True, out_dtype=torch.bfloat16)
        check(h1, qift.MNZ, x1, synth.had_block_for(K1), y1, a1, False)
        check(h2, qift.INT4, x2, synth.had_block_for(K2), y2, a2, False)
        check(h3, qift.POT, x3, synth.had_block_for(K3), y3, a3, True)
    clean()


def test_one_call_decodes_for_two_later_calls():
    # call 1 carries the decoding for calls 2 and 3 (other K, other level sets, five matrices in all); both then run on
    # ready levels; a list of more than eight matrices is refused
    M, K1, K2, K3 = 700, 512, 768, 256
    h1, g1 = make_weights(111, (520, 128), K1, qift.MNZ)
    h2, g2 = make_weights(121, (300, 136), K2, qift.INT4)
    h3, g3 = make_weights(131, (136, 136, 264), K3, qift.SYM)
    x1, _ = synth.activations(141, M, K1, 5)
    x2, _ = synth.activations(142, M, K2, 7)
    x3, _ = synth.activations(143, M, K3, 3)
    b1 = torch.full((qift.qift_levels_bytes(K1, g1),), 0x55, dtype=torch.uint8, device="cuda")
    b2 = torch.full((qift.qift_levels_bytes(K2, g2),), 0x55, dtype=torch.uint8, device="cuda")
    b3 = torch.full((qift.qift_levels_bytes(K3, g3),), 0x55, dtype=torch.uint8, device="cuda")
    y1, a1 = qift.qift_forward_multi(dev(x1), synth.had_block_for(K1), g1, qift.MNZ, CLIP, want_acc=True, levels_buf=b1,
                                     ahead=[(g2, K2, qift.INT4, b2), (g3, K3, qift.SYM, b3)])
    y2, a2 = qift.qift_forward_multi(dev(x2), synth.had_block_for(K2), g2, qift.INT4, CLIP, want_acc=True, levels_buf=b2, levels_ready=True)
    y3, a3 = qift.qift_forward_multi(dev(x3), synth.had_block_for(K3), g3, qift.SYM, CLIP, want_acc=True, levels_buf=b3, levels_ready=True)
    check(h1, qift.MNZ, x1, synth.had_block_for(K1), y1, a1, False)
    check(h2, qift.INT4, x2, synth.had_block_for(K2), y2, a2, False)
    check(h3, qift.SYM, x3, synth.had_block_for(K3), y3, a3, False)
    with pytest.raises(qift.QiftError) as e:
        qift.qift_forward_multi(dev(x1), synth.had_block_for(K1), g1, qift.MNZ, CLIP, levels_buf=b1,
                                ahead=[(g3, K3, qift.SYM, b3)] * 3)      # nine matrices
    assert e.value.status == qift.ERR_INVALID_ARG
    clean()


def test_forward_multi_rejects_bad_arguments():
    K, lv = 256, qift.MNZ
    host, gpu = make_weights(5, (128,), K, lv)
    x = dev(synth.activations(6, 600, K, 2)[0])
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(qift.QiftError) as e:       # M > 128 needs the levels buffer
        qift.qift_forward_multi(x, 256, gpu, lv, levels_buf=small)
    assert e.value.status == qift.ERR_WORKSPACE
    with pytest.raises(qift.QiftError) as e:       # scratch too small
        qift.qift_forward_multi(x, 256, gpu, lv, scratch=small)
    assert e.value.status == qift.ERR_WORKSPACE
    with pytest.raises(qift.QiftError) as e:       # five outputs
        qift.qift_forward_multi(x, 256, gpu * 5, lv)
    assert e.value.status == qift.ERR_INVALID_ARG
    with pytest.raises(qift.QiftError) as e:       # ahead buffer too small
        qift.qift_forward_multi(x, 256, gpu, lv, ahead=(gpu, K, lv, small))
    assert e.value.status == qift.ERR_WORKSPACE
    clean()


@pytest.mark.parametrize("M", [600, 24])
def test_linear_multi_on_a_quantized_activation(M):
    K, lv = 512, qift.SYM
    host, gpu = make_weights(61, (264, 520), K, lv)
    x, _ = synth.activations(62, M, K, 5)
    q_a, s_a = qift.qift_quantize_act(dev(x), 512, CLIP)
    ys, accs = qift.qift_linear_multi(q_a, s_a, gpu, lv, want_acc=True)
    check(host, lv, x, 512, ys, accs, False)
    clean()


def test_calibration_kernels_run_and_leave_the_status_clean():
    buf = torch.empty(64 << 20, dtype=torch.uint8, device="cuda").random_(0, 256)
    L = qift.lib()
    import ctypes
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert L.qift_calib_hbm_read(ctypes.c_void_p(buf.data_ptr()), buf.numel(), None, st) == qift.OK
    ops = ctypes.c_double(0.0)
    assert L.qift_calib_mma_i8(64, ctypes.byref(ops), st) == qift.OK
    assert ops.value == 2.0 * 256 * 256 * 128 * 64 * (torch.cuda.get_device_properties(0).multi_processor_count // 2)
    assert L.qift_calib_mma_i8(0, None, st) == qift.ERR_INVALID_ARG
    clean()
