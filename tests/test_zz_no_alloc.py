"""The workspace-free entry point rmm_score_select_static (GPU only; collected last on purpose).

It serves callers that cannot allocate device memory, so its scratch is a device array built into the library.
The test calls it through the C ABI twice in a row on different inputs and checks every output against the
regular entry point (rmm_score_select with a caller-provided workspace) bit for bit: the shared array keeps the
first call's contents, and the second call must not be disturbed by them.  A problem larger than the built-in
array must be refused with RMM_ERR_WORKSPACE before anything is launched.
"""
import pytest
import torch

import paper_2608_13426_b200 as rmm
from paper_2608_13426_b200 import binding, synth

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_entry_point_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    torch.cuda.set_device(0)
    cases = [(synth.heavy_tailed_activations(2048, 8192, seed=41).cuda(), 0.5),
             (synth.heavy_tailed_activations(777, 4096, seed=42).cuda(), 0.25)]
    for A, rho in cases:
        n = A.shape[1]
        k = rmm.rmm_keep_count(rho, n)
        # every buffer below belongs to the caller; the call under test gets no workspace
        idx = torch.full((k,), -1, dtype=torch.int32, device="cuda")
        energy = torch.zeros(n, dtype=torch.float32, device="cuda")
        retained = torch.zeros(1, dtype=torch.float32, device="cuda")
        rmm.rmm_score_select_static(A, idx, rho=rho, energy=energy, retained=retained)
        want_idx, _, want_energy, want_ret = rmm.rmm_score_select(A, rho=rho, want_energy=True, want_retained=True)
        torch.cuda.synchronize()
        assert torch.equal(idx, want_idx)
        assert torch.equal(energy, want_energy)
        assert torch.equal(retained, want_ret)
        assert rmm.rmm_score_select_static_status() == 0        # no kernel of this call reported an error
    # a batched problem that still fits
    Q = synth.gaussian((6, 300, 128), 1.0, seed=43).cuda()
    idx = torch.empty((6, 64), dtype=torch.int32, device="cuda")
    rmm.rmm_score_select_static(Q, idx, rho=0.5)
    want_idx, _, _, _ = rmm.rmm_score_select(Q, rho=0.5)
    torch.cuda.synchronize()
    assert torch.equal(idx, want_idx)


def test_static_scratch_rejects_oversize():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    torch.cuda.set_device(0)
    cap = rmm.rmm_score_select_static_capacity()
    assert cap == 4 << 20
    A = torch.zeros((64, 32, 16384), dtype=torch.bfloat16, device="cuda")      # energies alone: 64 * 16384 * 4 = 4 MiB
    idx = torch.full((64, 8192), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.RmmError) as e:
        rmm.rmm_score_select_static(A, idx, rho=0.5)
    assert e.value.code == binding.RMM_ERR_WORKSPACE and "built-in array" in str(e.value)
    torch.cuda.synchronize()
    assert int(idx.min()) == -7 and int(idx.max()) == -7                        # nothing was launched
    # the wrapper checks the caller's buffers before the call: a short idx would be written past its end
    small = torch.zeros((8, 64, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.RmmError) as e:
        rmm.rmm_score_select_static(small, torch.empty(100, dtype=torch.int32, device="cuda"), rho=0.5)
    assert e.value.code == binding.RMM_ERR_INVALID_ARG
