"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.
Index work (activation indices, scales, packed bytes) must be bit-exact; fp32 outputs must meet
relative L2 <= 2e-3 and max-abs <= 1e-2 * ||y_ref||_inf (the stated tolerance).  The kernels accumulate in
exact integers or fp32, for which the expected error is far smaller (derived bound: <= 1e-4 relative L2), so that
tighter bound is asserted as well."""
import numpy as np
import pytest
import torch

import paper_2506_12038_b200 as lcd
from oracle import lcd_oracle as O
from synth import gen

pytestmark = pytest.mark.gpu

REL_L2_TOL, MAXABS_TOL = 2e-3, 1e-2
TIGHT_REL_L2 = 1e-4


def check_y(y_gpu, y_ref, tight=True):
    y = y_gpu.detach().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(y))
    denom = np.linalg.norm(y_ref)
    rel = np.linalg.norm(y - y_ref) / (denom if denom > 0 else 1.0)
    mx = np.abs(y - y_ref).max()
    ninf = np.abs(y_ref).max()
    assert rel <= REL_L2_TOL, f"rel L2 {rel}"
    assert mx <= MAXABS_TOL * (ninf if ninf > 0 else 1.0), f"max abs {mx} vs {ninf}"
    if tight:
        assert rel <= TIGHT_REL_L2, f"rel L2 {rel} above the derived bound"
    # worst single token
    for m in range(y.shape[0]):
        d = np.linalg.norm(y_ref[m])
        if d > 0:
            assert np.linalg.norm(y[m] - y_ref[m]) / d <= REL_L2_TOL


# ------------------------------------------------------------------------------- input transformation
@pytest.mark.parametrize("M,K,ld_extra,use_inv", [(1, 4096, 0, True), (5, 1000, 0, True), (3, 999, 0, True),
                                                  (4, 264, 8, True), (2, 250, 3, False), (1, 1, 0, True),
                                                  (7, 11008, 0, True), (33, 520, 0, False),
                                                  # more than 296 tokens: the small-CTA instances, one per row-length bracket
                                                  (300, 520, 0, False), (300, 4096, 0, True), (301, 7000, 8, True),
                                                  (300, 11008, 0, True), (297, 13824, 0, True), (300, 17000, 0, True),
                                                  (300, 999, 0, True)])
def test_smooth_quantize_bit_exact(M, K, ld_extra, use_inv):
    ch = gen.outlier_channels(11, K, 0.01)
    x = gen.activations(100 + M + K, M, K, ch, 50.0)
    inv_s = (1.0 / (np.abs(gen.normal(5, K)) * 3 + 0.05)).astype(np.float32) if use_inv else None
    xd = torch.zeros((M, K + ld_extra), dtype=torch.float16, device="cuda")
    xd[:, :K] = torch.from_numpy(x).cuda()
    a, s = lcd.smooth_quantize_act(xd[:, :K], torch.from_numpy(inv_s).cuda() if use_inv else None)
    q_ref, s_ref = O.smooth_quantize(x, inv_s)
    assert np.array_equal(a.cpu().numpy(), O.pack_act(q_ref))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))


def test_smooth_quantize_edge_rows_and_static_mode():
    K = 512
    x = np.zeros((4, K), dtype=np.float16)
    x[1, 7] = 3.0                                   # a single non-zero
    x[2] = np.float16(1.0)                          # all equal
    x[3, ::2], x[3, 1::2] = np.float16(0.5), np.float16(-7.0)   # ties at +-0.5 after scaling
    a, s = lcd.smooth_quantize_act(torch.from_numpy(x).cuda())
    q_ref, s_ref = O.smooth_quantize(x, None)
    assert np.array_equal(a.cpu().numpy(), O.pack_act(q_ref)) and np.array_equal(s.cpu().numpy(), s_ref)
    assert s_ref[0] == 1.0 and not q_ref[0].any()
    # static mode (scale fixed offline): f = 1/(s_k*s_q) is given, a single multiply
    xs = (gen.normal(3, 4 * K).reshape(4, K) * 6).astype(np.float16)
    f = (1.0 / (np.abs(gen.normal(4, K)) + 0.5)).astype(np.float32)
    sq = torch.tensor([0.37], dtype=torch.float32, device="cuda")
    a2, s2 = lcd.smooth_quantize_act(torch.from_numpy(xs).cuda(), torch.from_numpy(f).cuda(), static_scale=sq)
    q2, sr2 = O.smooth_quantize(xs, f, static_scale=np.float32(0.37))
    assert np.array_equal(a2.cpu().numpy(), O.pack_act(q2)) and np.array_equal(s2.cpu().numpy(), sr2)
    assert q2.min() == -8 and q2.max() == 7


# ------------------------------------------------------------------------------- lookup + accumulation
def run_case(L, algo, tight=True):
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits, L.C))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    assert np.array_equal(a.cpu().numpy(), O.pack_act(q_ref))
    y = lcd.lut_linear(w, a, s, algo=algo)
    torch.cuda.synchronize()
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref), tight)
    return y


SHAPES = [(8, 256), (200, 1000), (1031, 520), (64, 4096), (24, 11008), (520, 2304)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("N,K", SHAPES)
@pytest.mark.parametrize("M", [1, 2, 3, 5, 16])
def test_register_lut_matches_oracle(bits, N, K, M):
    run_case(gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M), lcd.ALGO_REGISTER_LUT)


@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("N,K,M", [(8, 256, 1), (200, 1000, 2), (1031, 520, 5), (64, 4096, 8), (24, 11008, 16),
                                   (520, 2304, 11)])
def test_bucket_lut_matches_oracle(bits, N, K, M):
    # exact integer bucket sums dotted with the fp16 codebook in fp32: no fixed-point step at all
    run_case(gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M), lcd.ALGO_BUCKET_LUT)


@pytest.mark.parametrize("N,K", SHAPES + [(16, 256), (4096, 4096), (300, 28672), (11008, 512), (2050, 768)])
@pytest.mark.parametrize("fused", [False, True])
def test_shared_bucket_matches_oracle(N, K, fused):
    # one token, 2-bit indices: bucket tables in shared memory, column slices met in the scratch, which is left zero
    L = gen.random_case(seed=N + K + 77, N=N, K=K, bits=2, M=1)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 2))
    x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = torch.full((1, N), float("nan"), dtype=torch.float32, device="cuda")
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    if fused:
        fb = lcd.FusedBatch([(w, x, inv_s, y)], algo=lcd.ALGO_SHARED_BUCKET, status_word=word)
        for _ in range(2):
            fb.run()
        ws = fb.workspace
    else:
        a, s = lcd.smooth_quantize_act(x, inv_s)
        ws = torch.zeros((lcd.lut_linear_workspace_bytes(w, 1, lcd.ALGO_SHARED_BUCKET),), dtype=torch.uint8, device="cuda")
        for _ in range(2):
            lcd.lut_linear(w, a, s, y=y, algo=lcd.ALGO_SHARED_BUCKET, workspace=ws, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    assert not ws.any()
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))


def test_shared_bucket_grouped_fewer_centroids_and_refusals():
    shapes = [(200, 1000, 4), (4096, 512, 3), (24, 11008, 4), (1031, 520, 1), (8, 256, 2)]
    cases = [gen.random_case(seed=61 * i + 5, N=N, K=K, bits=2, M=1, C=C) for i, (N, K, C) in enumerate(shapes)]
    cases[1].x[0, :] = 0                                   # an all-zero token: scale 1, levels 0
    items, refs = [], []
    for L in cases:
        w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 2, L.C))
        y = torch.full((1, L.N), float("nan"), dtype=torch.float32, device="cuda")
        items.append((w, torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda(), y))
        q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
        refs.append(O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    fb = lcd.FusedBatch(items, algo=lcd.ALGO_SHARED_BUCKET, status_word=word)
    for _ in range(3):
        fb.run()
    torch.cuda.synchronize()
    assert int(word.item()) == 0 and not fb.workspace.any()
    for (w, x, inv_s, y), y_ref in zip(items, refs):
        check_y(y, y_ref)
    y0 = [it[3].clone() for it in items]
    fb.run()
    torch.cuda.synchronize()
    assert all(torch.equal(a, it[3]) for a, it in zip(y0, items))      # bit-identical from run to run
    # outside its range: more than one token, 3-bit indices
    L = gen.random_case(seed=3, N=64, K=512, bits=3, M=1)
    w3 = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 3))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    with pytest.raises(lcd.LcdError) as err:
        lcd.lut_linear(w3, a, s, algo=lcd.ALGO_SHARED_BUCKET)
    assert err.value.status == 2
    L = gen.random_case(seed=4, N=64, K=512, bits=2, M=2)
    w2 = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 2))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    with pytest.raises(lcd.LcdError) as err:
        lcd.lut_linear(w2, a, s, algo=lcd.ALGO_SHARED_BUCKET)
    assert err.value.status == 2


@pytest.mark.parametrize("bits,N,K,M", [(3, 40, 11008, 16), (2, 48, 28672, 8), (3, 16, 28672, 16), (2, 2064, 28672, 16),
                                        (3, 4096, 4096, 16)])
def test_lookup_with_column_panels(bits, N, K, M):
    # token count x row length too large for one shared-memory window: the columns are walked in panels and
    # every 16-row group is finished through the integer scratch
    L = gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M)
    run_case(L, lcd.ALGO_REGISTER_LUT)


@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("N,K", SHAPES + [(4096, 4096), (300, 28672)])
@pytest.mark.parametrize("M", [1, 3, 8, 16])
def test_tensor_core_lut_matches_oracle(bits, N, K, M):
    # the register-LUT tables and exact integer sums, looked-up bytes fed to tcgen05 kind::i8 through tensor memory;
    # row tiles whose columns are split over CTAs are finished through the integer scratch, which is left zero
    L = gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits, L.C))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    ws = torch.zeros((lcd.lut_linear_workspace_bytes(w, M, lcd.ALGO_TC_LUT),), dtype=torch.uint8, device="cuda")
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):
        lcd.lut_linear(w, a, s, y=y, algo=lcd.ALGO_TC_LUT, workspace=ws, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    assert not ws.any()
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))


@pytest.mark.parametrize("algo", ["register", "tensor"])
def test_grouped_launch_matches_oracle_and_leaves_scratch_zero(algo):
    algo = lcd.ALGO_REGISTER_LUT if algo == "register" else lcd.ALGO_TC_LUT
    shapes = [(2, 200, 1000, 1), (2, 4096, 512, 3), (2, 24, 11008, 5), (2, 1031, 520, 1), (2, 8, 256, 8)]
    for bits in (2, 3):
        cases = [gen.random_case(seed=31 * i + bits, N=N, K=K, bits=bits, M=M) for i, (_, N, K, M) in enumerate(shapes)]
        acts, items, refs = [], [], []
        for L in cases:
            w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, bits))
            x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
            a = torch.empty((L.M, w.K_pad // 2), dtype=torch.uint8, device="cuda")
            sc = torch.empty((L.M,), dtype=torch.float32, device="cuda")
            y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
            acts.append((x, inv_s, a, sc))
            items.append((w, a, sc, y))
            q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
            refs.append((q_ref, s_ref, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref)))
        qb, lb = lcd.ActBatch(acts), lcd.LinearBatch(items, algo=algo)
        for _ in range(3):          # repeated calls reuse the scratch the previous call left
            qb.run()
            lb.run()
        torch.cuda.synchronize()
        assert not lb.workspace.any()
        for (w, a, sc, y), (q_ref, s_ref, y_ref) in zip(items, refs):
            assert np.array_equal(a.cpu().numpy(), O.pack_act(q_ref))
            assert np.array_equal(sc.cpu().numpy(), s_ref)
            check_y(y, y_ref)


@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("N,K,M", [(128, 256, 32), (200, 1000, 17), (1031, 520, 40), (64, 4096, 100), (520, 2304, 256),
                                   (272, 768, 300), (1024, 1024, 513),
                                   (2560, 512, 2048), (9472, 256, 512),
                                   (4608, 1024, 1024),
                                   (4600, 1024, 1000)])    # ragged rows and tokens
@pytest.mark.parametrize("algo", ["int8", "fp16"])
def test_dense_tensor_core_path_matches_oracle(bits, N, K, M, algo):
    # int8: 16-bit fixed-point byte tables x integer levels, exact int32 sums (the default above 16 tokens);
    # fp16: fp16 centroids x integer levels, fp32 accumulation, only the order of the sums differs from the oracle
    algo = lcd.ALGO_DENSE_TC if algo == "int8" else lcd.ALGO_DENSE_F16
    L = gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M)
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits, L.C))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    lcd.lut_linear(w, a, s, y=y, algo=algo, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))
    if algo == lcd.ALGO_DENSE_TC:      # the default choice above 16 tokens is this path
        assert torch.equal(lcd.lut_linear(w, a, s), y)


@pytest.mark.parametrize("bits,N,K,M", [(2, 200, 11008, 17), (3, 72, 8192, 32), (2, 48, 28672, 25), (3, 40, 4096, 20)])
def test_between_17_and_32_tokens_library_choice_matches_oracle(bits, N, K, M):
    # LCD_ALGO_AUTO: on rows of at least 8192 columns two launches of the register-table kernel (16 tokens + the rest)
    # through one scratch, else the tensor-core kernel; the scratch is left zero either way
    L = gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, bits))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    ws = torch.zeros((max(lcd.lut_linear_workspace_bytes(w, M), 256),), dtype=torch.uint8, device="cuda")
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):
        lcd.lut_linear(w, a, s, y=y, workspace=ws, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    if K >= 8192:
        assert not ws.any()
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))


@pytest.mark.parametrize("N,K,M", [(200, 1000, 1), (4096, 4096, 1), (1031, 520, 8), (40, 11008, 16), (300, 28672, 4),
                                   (64, 2304, 20), (520, 768, 70), (24, 700, 300), (1031, 520, 40), (2560, 512, 2048),
                                   (4600, 1024, 1000)])
def test_four_bit_indices_library_choice_and_fused_launch(N, K, M):
    # 9 to 16 centroids per row (the paper's 3.3-bit point is 10): the byte tables hold sixteen entries (two
    # eight-entry lookups and a byte choice), in the register-table kernel up to 16 tokens and in the int8 tensor-core
    # kernel above.  Ten centroids, library's choice of kernel, and the one-launch form for up to 16 tokens.
    L = gen.random_case(seed=N + K + M + 4, N=N, K=K, bits=4, M=M, C=10)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 4, 10))
    x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
    a, s = lcd.smooth_quantize_act(x, inv_s)
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    y_ref = O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref)
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    ws = torch.zeros((max(lcd.lut_linear_workspace_bytes(w, M), 256),), dtype=torch.uint8, device="cuda")
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(2):
        lcd.lut_linear(w, a, s, y=y, workspace=ws, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    if M <= 16:
        assert not ws.any()            # (the tensor-core kernel keeps the expanded levels in its workspace)
    check_y(y, y_ref)
    if M <= 16:
        y2 = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        fb = lcd.FusedBatch([(w, x, inv_s, y2)], status_word=word)
        fb.run()
        torch.cuda.synchronize()
        assert int(word.item()) == 0 and torch.equal(y2, y)
    with pytest.raises(lcd.LcdError):                 # no one-hot bucket tables and no fp16-operand decoder at this width
        lcd.lut_linear(w, a, s, algo=lcd.ALGO_BUCKET_LUT if M <= 16 else lcd.ALGO_DENSE_F16)


def test_status_word_untouched_on_success():
    L = gen.random_case(seed=3, N=100, K=600, bits=2, M=2)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 2))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    word = torch.full((1,), 12345, dtype=torch.int32, device="cuda")
    lcd.lut_linear(w, a, s, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 12345


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("N,K,M", [(8, 256, 1), (200, 1000, 3), (1031, 520, 17), (64, 4096, 40), (24, 700, 33)])
def test_reference_kernel_matches_oracle(bits, N, K, M):
    run_case(gen.random_case(seed=N + K + M + bits, N=N, K=K, bits=bits, M=M), lcd.ALGO_REFERENCE)


@pytest.mark.parametrize("bits,C", [(3, 5), (3, 6), (2, 3), (2, 1), (3, 1), (4, 10), (4, 9), (4, 16), (4, 1)])
def test_fewer_centroids_than_index_width(bits, C):
    L = gen.random_case(seed=77 + C, N=40, K=777, bits=bits, M=2, C=C)
    run_case(L, lcd.ALGO_AUTO)
    run_case(L, lcd.ALGO_REFERENCE)


def test_shared_codebook_and_extreme_codebooks():
    # every row shares one codebook (the paper's per-layer codebook), a zero codebook, and fp16 extremes
    L = gen.random_case(seed=5, N=72, K=1280, bits=3, M=4)
    L.codebook[:] = L.codebook[0]
    run_case(L, lcd.ALGO_AUTO)
    L.codebook[:] = 0
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 3))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    assert not lcd.lut_linear(w, a, s).cpu().numpy().any()
    L.codebook[:] = np.array([60000, -60000, 6e-8, -6e-8, 1.0, -1.0, 0.0, 2.0 ** -14], dtype=np.float16)
    run_case(L, lcd.ALGO_AUTO, tight=True)


def test_deterministic_across_runs():
    L = gen.random_case(seed=9, N=256, K=4096, bits=2, M=1)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 2))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    y0 = lcd.lut_linear(w, a, s).clone()
    for _ in range(5):
        assert torch.equal(lcd.lut_linear(w, a, s), y0)


def test_host_buffer_entry_point():
    L = gen.random_case(seed=21, N=200, K=1000, bits=2, M=3)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 2))
    x_host = torch.from_numpy(L.x).pin_memory()
    y_host = torch.empty((3, 200), dtype=torch.float32).pin_memory()
    scratch = torch.zeros(lcd.linear_host_scratch_bytes(w, 3), dtype=torch.uint8, device="cuda")
    lcd.linear_host(w, x_host, torch.from_numpy(L.inv_s).cuda(), y_host, scratch)
    torch.cuda.synchronize()
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    check_y(y_host, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))


def test_grouped_host_buffer_entry_point():
    shapes = [(200, 1000, 1), (1031, 520, 3), (24, 11008, 5)]
    cases = [gen.random_case(seed=51 + i, N=N, K=K, bits=3, M=M) for i, (N, K, M) in enumerate(shapes)]
    ws = [lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, 3)) for L in cases]
    hb = lcd.HostBatch([(w, torch.from_numpy(L.inv_s).cuda(), L.M) for w, L in zip(ws, cases)])
    for _ in range(2):                      # the second call finds the scratch as the first one left it
        for i, L in enumerate(cases):
            hb.x_view(i).copy_(torch.from_numpy(L.x))
        hb.y_host.fill_(255)
        hb.run()
        torch.cuda.synchronize()
        for i, L in enumerate(cases):
            q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
            check_y(hb.y_view(i), O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))
    # the recorded form (what the benchmark's end-to-end leg replays): new inputs in the same pinned buffers
    hb.capture()
    for rep in range(2):
        for i, L in enumerate(cases):
            hb.x_view(i).copy_(torch.from_numpy(L.x) * (0.5 + rep))
        hb.y_host.fill_(255)
        hb.run()
        torch.cuda.synchronize()
        for i, L in enumerate(cases):
            q_ref, s_ref = O.smooth_quantize((L.x.astype(np.float32) * np.float32(0.5 + rep)).astype(np.float16), L.inv_s)
            check_y(hb.y_view(i), O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))


# ------------------------------------------------------------------------------- full sizes, bench launch shape
def _sampled_rows_check(L, y, q_ref, s_ref, n_rows=48, seed=0):
    rows = np.sort(gen.permutation(seed + L.N, L.N)[:n_rows])
    y_ref = O.lut_linear_rows(L.idx, L.codebook, q_ref, s_ref, rows)
    check_y(y[:, torch.from_numpy(rows).cuda()], y_ref)


_LAYER_CACHE = {}


def _config_layers(cfg_id, M):
    """The benchmark's inputs of one configuration (cached: generating a LLaMA-sized layer takes a minute).  Tokens
    are counter based, so the first M rows of a larger batch are the M-token batch itself."""
    cfg = gen.CONFIGS[cfg_id]
    big = max(cfg["Ms"])
    if cfg_id not in _LAYER_CACHE:
        _LAYER_CACHE[cfg_id] = [gen.make_layer(cfg_id, mi, N, K, cfg["bits"], big, outlier_frac=cfg["frac"],
                                               outlier_scale=cfg["scale"]) for mi, (_, N, K) in enumerate(cfg["shapes"])]
    out = []
    for L in _LAYER_CACHE[cfg_id]:
        import copy
        S = copy.copy(L)
        S.x, S.M = L.x[:M], M
        out.append(S)
    return out


def _all_rows_check(L, y, q_ref, s_ref):
    assert torch.isfinite(y).all()
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))


@pytest.mark.parametrize("cfg_id", [1, 4, 0])
def test_full_size_single_token_layer_fused_launch_all_rows(cfg_id):
    # The launch the benchmark times at one token: every projection of the layer in ONE lcd_linear_fused_batch call
    # (the kernel quantises x itself), library's choice of kernel, full sizes: the LLaMA-7B-shaped layer (2 bit), the
    # LLaMA-70B-shaped MLP (2 bit, 28672 x 8192 and 8192 x 28672) and the single 4096 x 4096 matrix (3 bit).  Every
    # output row is compared with the oracle; the launch runs twice on the scratch it left.
    cases = _config_layers(cfg_id, 1)
    items = []
    for L in cases:
        w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits))
        y = torch.full((1, L.N), float("nan"), dtype=torch.float32, device="cuda")
        items.append((w, torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda(), y))
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    fb = lcd.FusedBatch(items, status_word=word)
    for _ in range(2):
        fb.run()
    torch.cuda.synchronize()
    assert int(word.item()) == 0 and not fb.workspace.any()
    for L, (w, x, inv_s, y) in zip(cases, items):
        q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
        _all_rows_check(L, y, q_ref, s_ref)
    # the same launch replayed from a CUDA graph, as the benchmark does
    ys = [it[3].clone() for it in items]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        fb.run()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            fb.run()
            fb.run()
        for it in items:
            it[3].fill_(float("nan"))
        g.replay()
    torch.cuda.synchronize()
    assert int(word.item()) == 0 and not fb.workspace.any()
    assert all(torch.equal(a, it[3]) for a, it in zip(ys, items))


@pytest.mark.parametrize("cfg_id,M", [(1, 1), (2, 4), (2, 16), (4, 8)])
def test_full_size_layer_two_launches_all_rows(cfg_id, M):
    # The benchmark's other launch shape (more than one token, or --two-call): one grouped quantise launch and one
    # grouped lookup launch over the layer's projections, full sizes: the 7B-shaped layer at 2 bit (M = 1) and 3 bit
    # (M = 4, 16), the 70B-shaped MLP at M = 8.  Indices and scales bit for bit, every output row against the oracle.
    cases = _config_layers(cfg_id, M)
    acts, items = [], []
    for L in cases:
        w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits))
        x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
        a = torch.empty((M, w.K_pad // 2), dtype=torch.uint8, device="cuda")
        sc = torch.empty((M,), dtype=torch.float32, device="cuda")
        y = torch.full((M, L.N), float("nan"), dtype=torch.float32, device="cuda")
        acts.append((x, inv_s, a, sc))
        items.append((w, a, sc, y))
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    qb, lb = lcd.ActBatch(acts), lcd.LinearBatch(items, status_word=word)
    for _ in range(2):
        qb.run()
        lb.run()
    torch.cuda.synchronize()
    assert int(word.item()) == 0 and not lb.workspace.any()
    for L, (w, a, sc, y) in zip(cases, items):
        q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
        assert np.array_equal(a.cpu().numpy(), O.pack_act(q_ref))
        assert np.array_equal(sc.cpu().numpy(), s_ref)
        _all_rows_check(L, y, q_ref, s_ref)


@pytest.mark.parametrize("mi", [0, 4, 6])   # q 5120 x 5120 (192-token tiles), gate 13824 x 5120 (256-token tiles), down 5120 x 13824 (longest rows); 32 sampled rows each
def test_full_size_prefill_matrix_sampled_rows(mi):
    cfg = gen.CONFIGS[3]
    name, N, K = cfg["shapes"][mi]
    M = 2048
    L = gen.make_layer(3, mi, N, K, cfg["bits"], M, outlier_frac=cfg["frac"], outlier_scale=cfg["scale"])
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = lcd.lut_linear(w, a, s, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
    assert np.array_equal(a.cpu().numpy(), O.pack_act(q_ref))
    assert torch.isfinite(y).all()
    _sampled_rows_check(L, y, q_ref, s_ref, n_rows=32)


# ------------------------------------------------------------------------------- 8-bit activations (b = 8)
@pytest.mark.parametrize("M,K,ld_extra,use_inv", [(1, 256, 0, True), (3, 1000, 0, True), (5, 4096, 24, False),
                                                  (2, 250, 3, False), (1, 1, 0, True), (7, 11008, 0, True),
                                                  (300, 520, 0, False), (33, 264, 8, True)])
def test_smooth_quantize_8bit_bit_exact(M, K, ld_extra, use_inv):
    ch = gen.outlier_channels(11, K, 0.01)
    x = gen.activations(200 + M + K, M, K, ch, 50.0)
    inv_s = (1.0 / (np.abs(gen.normal(5, K)) * 3 + 0.05)).astype(np.float32) if use_inv else None
    xd = torch.zeros((M, K + ld_extra), dtype=torch.float16, device="cuda")
    xd[:, :K] = torch.from_numpy(x).cuda()
    a, s = lcd.smooth_quantize_act(xd[:, :K], torch.from_numpy(inv_s).cuda() if use_inv else None, act_bits=8)
    q_ref, s_ref = O.smooth_quantize(x, inv_s, act_bits=8)
    assert np.array_equal(a.cpu().numpy(), O.pad_act8(q_ref))
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))


def test_smooth_quantize_8bit_static_mode_reaches_minus_128():
    K = 512
    xs = (gen.normal(3, 4 * K).reshape(4, K) * 90).astype(np.float16)
    f = (1.0 / (np.abs(gen.normal(4, K)) + 0.5)).astype(np.float32)
    sq = torch.tensor([0.37], dtype=torch.float32, device="cuda")
    a, s = lcd.smooth_quantize_act(torch.from_numpy(xs).cuda(), torch.from_numpy(f).cuda(), static_scale=sq, act_bits=8)
    q, sr = O.smooth_quantize(xs, f, static_scale=np.float32(0.37), act_bits=8)
    assert np.array_equal(a.cpu().numpy(), O.pad_act8(q)) and np.array_equal(s.cpu().numpy(), sr)
    assert q.min() == -128 and q.max() == 127


ALGOS_ACT8 = {"reference": 1, "bucket": 2, "register": 3, "tensor": 6}


@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("N,K,M", [(8, 256, 1), (200, 1000, 2), (1031, 520, 5), (64, 4096, 8), (24, 11008, 16),
                                   (520, 2304, 11), (4096, 4096, 1), (48, 28672, 8)])
@pytest.mark.parametrize("algo", sorted(ALGOS_ACT8))
def test_lookup_with_8bit_levels_matches_oracle(bits, N, K, M, algo):
    # the same kernels with signed-byte levels: only the staging of the token operand differs
    L = gen.random_case(seed=N + K + M + bits + 8, N=N, K=K, bits=bits, M=M)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits, L.C))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda(), act_bits=8)
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s, act_bits=8)
    assert np.array_equal(a.cpu().numpy(), O.pad_act8(q_ref))
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.zeros((max(lcd.lut_linear_workspace_bytes(w, M, ALGOS_ACT8[algo]), 256),), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        lcd.lut_linear(w, a, s, y=y, algo=ALGOS_ACT8[algo], workspace=ws, status_word=word)
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    if algo != "reference":
        assert not ws.any()
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref), tight=algo != "reference")


@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("N,K,M", [(128, 256, 32), (200, 1000, 17), (1031, 520, 40), (520, 2304, 256),
                                   (1024, 1024, 513), (4600, 1024, 1000)])
def test_dense_path_with_8bit_levels_matches_oracle(bits, N, K, M):
    L = gen.random_case(seed=N + K + M + bits + 8, N=N, K=K, bits=bits, M=M)
    w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits, L.C))
    a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda(), act_bits=8)
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    lcd.lut_linear(w, a, s, y=y, status_word=word)           # AUTO: the int8 tensor-core kernel above 16 tokens
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s, act_bits=8)
    assert np.array_equal(a.cpu().numpy(), O.pad_act8(q_ref))
    check_y(y, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))
    with pytest.raises(lcd.LcdError):                          # the fp16-operand kernel takes 4-bit levels only
        lcd.lut_linear(w, a, s, y=y, algo=lcd.ALGO_DENSE_F16)


@pytest.mark.parametrize("algo", ["register", "tensor"])
def test_grouped_launch_with_8bit_levels(algo):
    algo = lcd.ALGO_REGISTER_LUT if algo == "register" else lcd.ALGO_TC_LUT
    shapes = [(200, 1000, 1), (4096, 512, 3), (24, 11008, 5), (1031, 520, 1), (8, 256, 8)]
    for bits in (2, 3):
        cases = [gen.random_case(seed=37 * i + bits, N=N, K=K, bits=bits, M=M) for i, (N, K, M) in enumerate(shapes)]
        acts, items, refs = [], [], []
        for L in cases:
            w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, bits))
            x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
            a = torch.empty((L.M, w.K_pad), dtype=torch.int8, device="cuda")
            sc = torch.empty((L.M,), dtype=torch.float32, device="cuda")
            y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
            acts.append((x, inv_s, a, sc))
            items.append((w, a, sc, y))
            q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s, act_bits=8)
            refs.append((q_ref, s_ref, O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref)))
        word = torch.zeros((1,), dtype=torch.int32, device="cuda")
        qb, lb = lcd.ActBatch(acts), lcd.LinearBatch(items, algo=algo, status_word=word)
        for _ in range(2):
            qb.run()
            lb.run()
        torch.cuda.synchronize()
        assert int(word.item()) == 0 and not lb.workspace.any()
        for (w, a, sc, y), (q_ref, s_ref, y_ref) in zip(items, refs):
            assert np.array_equal(a.cpu().numpy(), O.pad_act8(q_ref))
            assert np.array_equal(sc.cpu().numpy(), s_ref)
            check_y(y, y_ref)


# ------------------------------------------------------------------------------- steps 1+2+3 in one launch
@pytest.mark.parametrize("bits", [2, 3])
@pytest.mark.parametrize("algo", ["register", "bucket"])
def test_fused_launch_equals_two_call_path_and_oracle(bits, algo):
    # the lookup kernel quantises x itself: same binary32 steps, so y must equal the two-call result bit for bit
    algo = lcd.ALGO_REGISTER_LUT if algo == "register" else lcd.ALGO_BUCKET_LUT
    shapes = [(200, 1000, 1), (4096, 512, 3), (24, 11008, 5), (1031, 520, 1), (8, 256, 8), (40, 250, 2),   # 250: unaligned rows
              (48, 28672, 16)]                                                                           # column panels
    cases = [gen.random_case(seed=41 * i + bits, N=N, K=K, bits=bits, M=M) for i, (N, K, M) in enumerate(shapes)]
    cases[0].x[0, :] = 0                                    # an all-zero token: scale 1, levels 0
    items, two_call, refs = [], [], []
    for L in cases:
        w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, bits))
        x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
        y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
        items.append((w, x, inv_s, y))
        a, s = lcd.smooth_quantize_act(x, inv_s)
        two_call.append(lcd.lut_linear(w, a, s, algo=algo))
        q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
        refs.append(O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    fb = lcd.FusedBatch(items, algo=algo, status_word=word)
    for _ in range(2):
        fb.run()
    torch.cuda.synchronize()
    assert int(word.item()) == 0 and not fb.workspace.any()
    for (w, x, inv_s, y), y2, y_ref in zip(items, two_call, refs):
        assert torch.equal(y, y2)
        check_y(y, y_ref)
    # without smoothing factors
    w, x, _, y = items[3]
    fb1 = lcd.FusedBatch([(w, x, None, y)], algo=algo)
    fb1.run()
    a, s = lcd.smooth_quantize_act(x, None)
    assert torch.equal(y, lcd.lut_linear(w, a, s, algo=algo))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_fused_call_with_many_tokens_equals_two_call_path_and_oracle(bits):
    # more than 16 tokens: one transformation launch for all problems writes the tensor-core kernel's signed bytes
    # directly; the levels are the same, so y equals the two-call result bit for bit
    shapes = [(200, 1000, 33), (130, 520, 64), (24, 11008, 300), (257, 250, 40), (1031, 4096, 130), (72, 768, 17)]   # 250: unaligned rows
    C = 10 if bits == 4 else None
    cases = [gen.random_case(seed=71 * i + bits, N=N, K=K, bits=bits, M=M, C=C) for i, (N, K, M) in enumerate(shapes)]
    cases[1].x[3, :] = 0                                    # an all-zero token: scale 1, levels 0
    items, two_call, refs = [], [], []
    for L in cases:
        w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, bits, C) if C else lcd.pack_weights(L.idx, L.codebook, bits))
        x, inv_s = torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda()
        y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
        items.append((w, x, inv_s, y))
        a, s = lcd.smooth_quantize_act(x, inv_s)
        two_call.append(lcd.lut_linear(w, a, s, algo=lcd.ALGO_DENSE_TC))
        q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
        refs.append(O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref))
    word = torch.zeros((1,), dtype=torch.int32, device="cuda")
    fb = lcd.FusedBatch(items, status_word=word)
    for _ in range(2):
        fb.run()
    torch.cuda.synchronize()
    assert int(word.item()) == 0
    for (w, x, inv_s, y), y2, y_ref in zip(items, two_call, refs):
        assert torch.equal(y, y2)
        check_y(y, y_ref)
    # a mix of few and many tokens is refused before anything is launched
    with pytest.raises(lcd.LcdError) as err:
        lcd.FusedBatch([items[0], (items[0][0], items[0][1][:4], items[0][2], items[0][3][:4])])
    assert err.value.status == 2


# ------------------------------------------------------------------------------- adaptive smoothing search (offline)
@pytest.mark.parametrize("T,K,ld_extra", [(128, 4096, 0), (64, 1000, 8), (5, 250, 3), (1, 256, 0)])
def test_smoothing_search_matches_oracle(T, K, ld_extra):
    ch = gen.outlier_channels(7, K, 0.01)
    x = gen.activations(900 + T + K, T, K, ch, 50.0)
    wmax = (np.abs(gen.normal(8, K)) * 0.05 + 0.01).astype(np.float32)
    wmax[3 % K] = 0.0                                        # a dead weight column keeps s = 1
    alphas = [0.0, 0.2, 0.35, 0.5, 0.65, 0.8, 1.0]
    xd = torch.zeros((T, K + ld_extra), dtype=torch.float16, device="cuda")
    xd[:, :K] = torch.from_numpy(x).cuda()
    best, mse, inv = lcd.smoothing_search(xd[:, :K], torch.from_numpy(wmax).cuda(), alphas)
    torch.cuda.synchronize()
    b_ref, mse_ref = O.smoothing_search(x, wmax, alphas)
    # binary64 powers from two libraries may round a factor to neighbouring binary32 values; a level of that channel
    # that sat on a rounding tie then flips, which changes its squared error only in second order: observed 4e-7 of
    # the mean on 128 x 4096 and 4e-6 on 5 x 250 (one flip among 1250 values); the sums themselves agree to 1e-11
    np.testing.assert_allclose(mse.cpu().numpy(), mse_ref, rtol=1e-4, atol=0)
    np.testing.assert_allclose(mse.cpu().numpy()[[0, -1]], mse_ref[[0, -1]], rtol=1e-11, atol=0)   # alpha 0 and 1: exact powers
    assert int(best.item()) == b_ref
    s_ref = O.smoothing_factors(np.abs(x.astype(np.float64)).max(axis=0), wmax, alphas[b_ref])
    inv_ref = (np.float32(1.0) / s_ref).astype(np.float32)
    # the powers are binary64 on both sides but from different libraries: s may differ in its last binary32 bit,
    # its reciprocal then by up to three
    got = inv.cpu().numpy()
    assert np.all(np.abs(got.view(np.int32).astype(np.int64) - inv_ref.view(np.int32).astype(np.int64)) <= 3)
    # the chosen factors feed the online transformation unchanged
    a, sc = lcd.smooth_quantize_act(xd[:, :K], inv, act_bits=8)
    q_ref, s_q_ref = O.smooth_quantize(x, got, act_bits=8)
    assert np.array_equal(a.cpu().numpy(), O.pad_act8(q_ref)) and np.array_equal(sc.cpu().numpy(), s_q_ref)


# ------------------------------------------------------------------------------- reclassification (offline)
@pytest.mark.parametrize("N,K,C,ld_extra", [(64, 4096, 4, 0), (33, 1000, 8, 8), (5, 250, 5, 3), (3, 7, 1, 0), (2, 300, 16, 0)])
def test_reclassify_matches_oracle(N, K, C, ld_extra):
    cb = np.sort(gen.normal(50 + N, N * C).reshape(N, C), axis=1).astype(np.float16)
    idx = (gen.permutation(51 + K, N * K) % C).astype(np.uint8).reshape(N, K)
    dw = (gen.normal(52 + C, N * K).reshape(N, K) * 0.4).astype(np.float32)
    dw[0, :min(K, 4)] = 0.0
    dwd = torch.zeros((N, K + ld_extra), dtype=torch.float32, device="cuda")
    dwd[:, :K] = torch.from_numpy(dw).cuda()
    new_idx, dC, cnt = lcd.reclassify(torch.from_numpy(idx).cuda(), torch.from_numpy(cb).cuda(), dwd[:, :K])
    torch.cuda.synchronize()
    r_idx, r_dC, r_cnt = O.reclassify(idx, cb, dw)
    assert np.array_equal(new_idx.cpu().numpy(), r_idx)                    # decisions: bit-exact
    assert np.array_equal(cnt.cpu().numpy().astype(np.int64), r_cnt)
    np.testing.assert_allclose(dC.cpu().numpy(), r_dC, rtol=1e-11, atol=1e-11)   # binary64 sums in another order


# ------------------------------------------------------------------------------- DBCI (offline)
def _dbci_inputs(case):
    if case == "gauss":                      # a layer's weights: N(0, 0.02) with a few outliers
        w = gen.normal(71, 200000) * 0.02
        w[::20000] *= 12
    elif case == "clumps":
        w = np.concatenate([gen.normal(72, 3000) * 0.02, 0.1 + gen.normal(73, 250) * 0.001,
                            -0.08 + gen.normal(74, 150) * 0.001, [-0.5, -0.49, -0.495, 0.6, 0.61, 0.605]])
    elif case == "tiny":
        w = np.array([-10.0, -1.0, -0.9, -1.1, 1.0, 1.1, 0.9, 1.05, 12.0])
    elif case == "one_sided":                # no negative weights at all
        w = np.abs(gen.normal(75, 5000)) * 0.02 + 0.001
    else:                                    # "single"
        w = np.array([0.25])
    return w.astype(np.float32)


@pytest.mark.parametrize("case", ["gauss", "clumps", "tiny", "one_sided", "single"])
def test_dbci_matches_oracle(case):
    w = _dbci_inputs(case)
    r = lcd.dbci(torch.from_numpy(w).cuda(), max_centroids=4096)
    torch.cuda.synchronize()
    # the plain oracle is quadratic: the 200000-weight case takes its n log n form, which a CPU test holds to the
    # plain one
    ref = O.dbci_scan(w) if w.size > 20000 else O.dbci(w)
    assert np.array_equal(r["sorted"].cpu().numpy(), ref["sorted"])
    assert r["sigma"] == ref["sigma"] and r["eps"] == ref["eps"]            # binary64 scalars: identical operations
    assert (r["min_pts"], r["left"], r["right"]) == (ref["min_pts"], ref["left"], ref["right"])
    assert np.array_equal(r["labels"].cpu().numpy().astype(np.int64), ref["labels"])
    assert r["n_noise"] == int((ref["labels"] < 0).sum())
    assert np.array_equal(r["centroids"].cpu().numpy().astype(np.float64), ref["centroids"])
