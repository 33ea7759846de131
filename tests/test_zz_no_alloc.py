"""dlm_unmask_select_static, the entry point for callers that may not allocate device memory
(hosts running under a fixed memory plan, plug-ins without an allocator of their own): it
takes no context and no workspace, its scratch is an array inside the library.  Its results
must equal those of dlm_unmask_select bit for bit, also on a second call that reuses the
array with other contents, and both must agree with the CPU oracle.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2505_21467_b200 as dlm
from workloads import make_logits, make_mask
from helpers import CONF_RTOL, Dev, gpu_unmask, topk_margin

pytestmark = pytest.mark.gpu


def _static(logits, masked, tokens, k):
    B, Lblk, V = logits.shape
    tok = torch.full((B, Lblk), -9, dtype=torch.int32, device="cuda")
    conf = torch.full((B, Lblk), float("nan"), device="cuda")
    sel_idx = torch.full((B, k), -9, dtype=torch.int32, device="cuda")
    n_sel = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    dlm.dlm_unmask_select_static(logits, B, Lblk, V, masked, tokens, k, tok, conf, sel_idx, n_sel)
    return tok, conf, sel_idx, n_sel


def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row(oracle):
    dev = Dev()
    checked_against_oracle = 0
    # two different shapes back to back: the second call finds the first call's partials in the array
    for B, Lblk, V, n_masked, k, seed in ((2, 32, 20001, 20, 4, 71), (3, 48, 9000, 48, 5, 72)):
        logits = make_logits(B, Lblk, V, (1.0, 8.0), seed, device="cuda")
        masked0 = make_mask(B, Lblk, n_masked, seed).cuda()
        m_a, t_a = masked0.clone(), torch.full((B, Lblk), -1, dtype=torch.int32, device="cuda")
        m_b, t_b = masked0.clone(), t_a.clone()
        want = gpu_unmask(dev, logits, m_a, t_a, k)
        got = _static(logits, m_b, t_b, k)
        torch.cuda.synchronize()
        assert dev.status() == 0
        for w, g in zip(want, got):
            assert torch.equal(w, g)
        assert torch.equal(m_a, m_b) and torch.equal(t_a, t_b)
        assert int(got[3].min()) == min(k, n_masked)
        # and against the CPU oracle, so that the check does not rest on the CUDA path alone: token ids, selected
        # positions, masks and tokens bit for bit, confidences within the tolerance of the fp32 sums
        o_m, o_t = masked0.cpu().numpy().copy(), np.full((B, Lblk), -1, np.int32)
        o_tok, o_conf, o_sel, o_n = oracle.unmask_select(logits.cpu().numpy(), o_m, o_t, k)
        if topk_margin(o_conf, masked0.cpu().numpy(), k) > 1e-4:   # else several top-k sets are acceptable
            np.testing.assert_array_equal(got[2].cpu().numpy(), o_sel)
            np.testing.assert_array_equal(got[3].cpu().numpy(), o_n)
            np.testing.assert_array_equal(m_b.cpu().numpy(), o_m)
            np.testing.assert_array_equal(t_b.cpu().numpy(), o_t)
            checked_against_oracle += 1
        np.testing.assert_array_equal(got[0].cpu().numpy(), o_tok)
        on = masked0.cpu().numpy().astype(bool)
        np.testing.assert_allclose(got[1].cpu().numpy()[on], o_conf[on], rtol=CONF_RTOL)
    assert checked_against_oracle >= 1


def test_static_scratch_rejects_sizes_beyond_its_array():
    B, Lblk, V = 60, 1024, 8192          # 60 * 1024 rows x 2 chunks = 122880 partials > 65536
    z = torch.zeros(1, dtype=torch.float32, device="cuda")
    m = torch.zeros(1, dtype=torch.uint8, device="cuda")
    i = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(dlm.DlmError) as e:
        dlm.dlm_unmask_select_static(z, B, Lblk, V, m, i, 1, i, z, i, i)
    assert e.value.code == dlm.DLM_ERR_WORKSPACE
