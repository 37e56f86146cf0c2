"""lcd_lut_linear_static: the M <= 16 lookup for callers that cannot allocate device memory (a plug-in inside
an application that owns the memory pool, a serving loop that may not call cudaMalloc once it is running).
Its scratch is a fixed array inside the library, shared by every call, so the test runs it twice in a row on
different layers and compares each result with lcd_lut_linear, which uses a workspace the caller allocated.
This file is collected last on purpose: a failure here leaves every other test already run."""
import numpy as np
import pytest
import torch

import paper_2506_12038_b200 as lcd
from oracle import lcd_oracle as O
from paper_2506_12038_b200 import binding
from synth import gen

pytestmark = pytest.mark.gpu

REL_L2_TOL, MAXABS_TOL = 2e-3, 1e-2       # the tolerance of the parity tests


def _close(y, y_ref):
    y, y_ref = y.double().cpu().numpy(), y_ref.double().cpu().numpy()
    assert np.all(np.isfinite(y))
    rel = np.linalg.norm(y - y_ref) / max(np.linalg.norm(y_ref), 1e-30)
    assert rel <= REL_L2_TOL, rel
    assert np.abs(y - y_ref).max() <= MAXABS_TOL * max(np.abs(y_ref).max(), 1e-30)


@pytest.mark.parametrize("algo", [lcd.ALGO_AUTO, lcd.ALGO_BUCKET_LUT])
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row(algo):
    # second case: token count x row length too large for one activation window, so every 16-row group is
    # finished through the scratch; it runs right after the first one on what that call left behind
    cases = [gen.random_case(seed=41, N=520, K=2304, bits=2, M=3), gen.random_case(seed=42, N=40, K=11008, bits=3, M=16)]
    outs, oracle = [], []
    for L in cases:
        w = lcd.PackedWeights(lcd.pack_weights(L.idx, L.codebook, L.bits))
        a, s = lcd.smooth_quantize_act(torch.from_numpy(L.x).cuda(), torch.from_numpy(L.inv_s).cuda())
        y_ref = lcd.lut_linear(w, a, s, algo=algo)
        y = torch.full((L.M, L.N), float("nan"), dtype=torch.float32, device="cuda")
        outs.append((lcd.lut_linear_static(w, a, s, y, algo=algo), y_ref, w, a, s))
        q_ref, s_ref = O.smooth_quantize(L.x, L.inv_s)
        oracle.append(torch.from_numpy(O.lut_linear_dequant(L.idx, L.codebook, q_ref, s_ref)))
    torch.cuda.synchronize()
    for (y, y_ref, *_), y_cpu in zip(outs, oracle):
        _close(y, y_ref)          # the entry point with a caller-allocated workspace
        _close(y, y_cpu)          # and the CPU oracle
    # the same layer again: identical bits (the sums are integers, the order of arrival does not matter)
    y, y_ref, w, a, s = outs[0]
    y2 = torch.empty_like(y)
    # what the entry point is for: the call itself obtains no device memory, neither from torch's pool nor from the
    # driver (the first calls above have looked the array's address up already)
    torch.cuda.synchronize()
    count = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]      # allocations made so far, ever
    made_before, (free_before, _) = count(), torch.cuda.mem_get_info()
    lcd.lut_linear_static(w, a, s, y2, algo=algo)
    torch.cuda.synchronize()
    assert count() == made_before
    assert torch.cuda.mem_get_info()[0] >= free_before
    assert torch.equal(y2, y)


def test_static_scratch_refuses_layers_beyond_its_size():
    # 70000 rows need more integer scratch than the built-in array holds: refused before anything is enqueued
    N, K = 70000, 256
    idx = np.zeros((N, K), dtype=np.uint8)
    w = lcd.PackedWeights(lcd.pack_weights(idx, np.zeros((N, 4), dtype=np.float16), 2))
    # (asked of the register-table family, which is what the entry point runs for LCD_ALGO_AUTO)
    assert lcd.lut_linear_workspace_bytes(w, 1, lcd.ALGO_REGISTER_LUT) > binding.STATIC_SCRATCH_BYTES
    a = torch.zeros((1, 128), dtype=torch.uint8, device="cuda")
    s = torch.ones((1,), dtype=torch.float32, device="cuda")
    y = torch.zeros((1, N), dtype=torch.float32, device="cuda")
    with pytest.raises(lcd.LcdError) as err:
        lcd.lut_linear_static(w, a, s, y)
    assert err.value.status == 3      # LCD_ERR_BUFFER_TOO_SMALL
    with pytest.raises(lcd.LcdError) as err:
        lcd.lut_linear_static(w, torch.zeros((17, 128), dtype=torch.uint8, device="cuda"),
                              torch.ones((17,), dtype=torch.float32, device="cuda"),
                              torch.zeros((17, N), dtype=torch.float32, device="cuda"))
    assert err.value.status == 2      # LCD_ERR_UNSUPPORTED
