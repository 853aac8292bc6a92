"""Helpers shared by the GPU parity tests (imported only when a GPU test runs)."""
import numpy as np
import torch

from oracle import gva_oracle as orc
from paper_2609_13285_b200 import binding as gb
from paper_2609_13285_b200 import build as gbuild
from paper_2609_13285_b200 import harness

# Tolerances against the fp64 oracle (which reads the identical stored cache values, so cache
# rounding is not an error source):
#   contract   : max-abs <= 2e-2 (bf16 cache, f32 accumulate), <= 1e-5 (f32 cache)
#   tight gates: f32 arithmetic on exact cache values -> max-abs <= 2e-5 and rel-L2 <= 1e-5
TOL_F32_CACHE = 1e-5
TOL_BF16_CONTRACT = 2e-2
TOL_TIGHT_MAXABS = 2e-5
TOL_TIGHT_REL_L2 = 1e-5
TOL_QABS = 1e-5


def ensure_built():
    gbuild.build()
    gb.load()


def kernels_for(case):
    """Kernel variants a case can run on."""
    ks = [gb.GVA_KERNEL_FMA]
    if case.cache_dtype == "bf16":
        ks.append(gb.GVA_KERNEL_MMA)
    return ks


def rel_l2(a, ref):
    d = np.linalg.norm((a - ref).ravel())
    n = np.linalg.norm(ref.ravel())
    return d / n if n > 0 else d


def oracle_for_gpu_q(case, q_abs_dev, seq_lens=None):
    """Oracle decode fed with the absorbed query the GPU actually uses (f32 widened to f64)."""
    q = q_abs_dev.detach().cpu().numpy().astype(np.float64)
    return orc.decode_case(case, q, seq_lens=seq_lens)


def check_decode(case, kernel, num_splits=0, tight=True, dc=None):
    own = dc is None
    if own:
        dc = harness.upload(case, kernel=kernel)
    try:
        dc.absorb()
        dc.out.fill_(float("nan"))
        dc.lse.fill_(float("nan"))
        out, lse = dc.decode(num_splits=num_splits)
        torch.cuda.synchronize()
        assert int(dc.status.item()) == 0, f"device status {int(dc.status.item()):#x}"
        ref_out, ref_lse = oracle_for_gpu_q(case, dc.q_abs)
        o = out.cpu().numpy().astype(np.float64)
        l = lse.cpu().numpy().astype(np.float64)
        assert np.isfinite(o).all(), "non-finite output"
        err = float(np.max(np.abs(o - ref_out))) if o.size else 0.0
        contract = TOL_F32_CACHE if case.cache_dtype == "f32" else TOL_BF16_CONTRACT
        assert err <= contract, f"max-abs {err:.3e} > contract {contract}"
        if tight:
            assert err <= TOL_TIGHT_MAXABS, f"max-abs {err:.3e} > tight gate"
            assert rel_l2(o, ref_out) <= TOL_TIGHT_REL_L2, f"rel-L2 {rel_l2(o, ref_out):.3e}"
        live = np.asarray(case.seq_lens) > 0
        if live.any():
            assert np.max(np.abs(l[live] - ref_lse[live])) <= 1e-4 * max(1.0, np.max(np.abs(ref_lse[live])))
        if (~live).any():
            assert np.all(o[~live] == 0) and np.all(np.isneginf(l[~live]))
        return err
    finally:
        if own:
            dc.close()
