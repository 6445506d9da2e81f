"""Shared helpers for the GPU parity tests: error measures and a paired runner that
feeds identical seeded inputs to the CUDA library (through its C ABI) and to the
CPU float64 oracle."""
from __future__ import annotations

import numpy as np

from paper_2307_02047_b200 import synth

# Tolerances: max error <= 1e-5 after one step and <= 1e-4 after ten steps (fp32 state).
TOL_STEP1 = 1e-5
TOL_STEP10 = 1e-4


def err_signed(x: np.ndarray, ref: np.ndarray) -> float:
    """For p and m (signed, cancelling): max |x - ref| / (|ref| + RMS(ref))."""
    ref = ref.astype(np.float64)
    rms = float(np.sqrt(np.mean(ref * ref)))
    den = np.abs(ref) + rms
    den[den == 0.0] = 1.0
    return float(np.max(np.abs(x.astype(np.float64) - ref) / den))


def err_strict(x: np.ndarray, ref: np.ndarray) -> float:
    """Strict element-wise relative error max |x - ref| / |ref| (reported, never gated: for a
    signed quantity that cancels, some element of 1e8 is always close to zero)."""
    ref = ref.astype(np.float64)
    nz = ref != 0.0
    if not nz.any():
        return 0.0
    return float(np.max(np.abs(x.astype(np.float64)[nz] - ref[nz]) / np.abs(ref[nz])))


def err_update(p: np.ndarray, p_ref: np.ndarray, p0: np.ndarray, steps: int) -> float:
    """Error of the cumulative update theta_t - theta_0 against the oracle's, measured on the
    scale of the update itself: max |d - d_ref| / (|d_ref| + RMS(d_ref)).

    theta moves by ~1e-3 per step while |theta| ~ 0.02, so the gate on theta alone is about
    ten times less sensitive to the last line of Algorithm 2 than this one.  theta is stored
    in fp32, and every step rounds it once (at most half an ulp, <= 2^-24 * 2|theta|), whatever
    the implementation; that unavoidable storage rounding, steps * 2^-23 * |theta|, is taken
    off the difference before it is compared, so that only the arithmetic is judged."""
    p_ref = p_ref.astype(np.float64)
    p0 = p0.astype(np.float64)
    d = p.astype(np.float64) - p0
    d_ref = p_ref - p0
    rms = float(np.sqrt(np.mean(d_ref * d_ref)))
    den = np.abs(d_ref) + rms
    den[den == 0.0] = 1.0
    storage = steps * (2.0 ** -23) * np.abs(p_ref)
    return float(np.max(np.maximum(np.abs(d - d_ref) - storage, 0.0) / den))


def err_positive(x: np.ndarray, ref: np.ndarray) -> float:
    """For the positive reductions r, c, R, C (and vector v, S): strict element-wise relative error."""
    ref = ref.astype(np.float64)
    x = x.astype(np.float64)
    zero = ref == 0.0                      # untouched state (e.g. S of a no-confidence vector)
    if np.any(x[zero] != 0.0):
        return float("inf")
    if zero.all():
        return 0.0
    return float(np.max(np.abs(x[~zero] - ref[~zero]) / ref[~zero]))


def to_torch_grad(torch, g: np.ndarray, device):
    if g.dtype == np.uint16:
        return torch.from_numpy(g.view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(g).to(device)


def gate(res: dict, label: str = "", tol_of=None) -> None:
    """Assert every gated error of a run_paired result: 1e-5 at step 1, 1e-4 at any later
    step.  Entries named strict_* are information only (see err_strict)."""
    assert res
    if label:
        print("PARITY", label, {k: {n: float("%.3g" % e) for n, e in v.items()} for k, v in res.items()})
    for step, worst in res.items():
        tol = (TOL_STEP1 if step == 1 else TOL_STEP10) if tol_of is None else tol_of(step)
        for name, e in worst.items():
            if name.startswith("strict_"):
                continue
            assert e <= tol, f"{label} step {step}: {name} error {e:.3e} > {tol:.0e}  ({worst})"


def compare_state(opt, orc, indices=None, p0=None, steps: int = 1) -> dict:
    """Worst error per state name between a CameOptimizer and an OracleOptimizer.

    ``p0`` (the initial parameters of the compared tensors, in the oracle's order) adds the
    gate on the cumulative update, ``dp``."""
    worst = dict(p=0.0, m=0.0, r=0.0, c=0.0, R=0.0, C=0.0, strict_p=0.0, strict_m=0.0)
    if p0 is not None:
        worst["dp"] = 0.0
    idx = range(len(opt.params)) if indices is None else indices
    for k, i in enumerate(idx):
        j = i if indices is None else k
        for a in (opt.params[i], opt.m[i]):
            assert bool(a.isfinite().all()), "non-finite value in GPU state"
        p_gpu, m_gpu = opt.params[i].cpu().numpy(), opt.m[i].cpu().numpy()
        worst["p"] = max(worst["p"], err_signed(p_gpu, orc.p[j]))
        worst["m"] = max(worst["m"], err_signed(m_gpu, orc.m[j]))
        worst["strict_p"] = max(worst["strict_p"], err_strict(p_gpu, orc.p[j]))
        worst["strict_m"] = max(worst["strict_m"], err_strict(m_gpu, orc.m[j]))
        if p0 is not None:
            worst["dp"] = max(worst["dp"], err_update(p_gpu, orc.p[j], p0[j], steps))
        worst["r"] = max(worst["r"], err_positive(opt.r[i].cpu().numpy(), orc.r[j]))
        worst["R"] = max(worst["R"], err_positive(opt.R[i].cpu().numpy(), orc.R[j]))
        if opt.c[i] is not None:
            worst["c"] = max(worst["c"], err_positive(opt.c[i].cpu().numpy(), orc.c[j]))
            worst["C"] = max(worst["C"], err_positive(opt.C[i].cpu().numpy(), orc.C[j]))
    return worst


def run_paired(torch, binding, oracle, w: synth.Workload, seed: int, steps: int, check_at,
               flags=None, hparams=None, device="cuda:0", oracle_idx=None, workers: int = 0,
               algorithm: str = "came", bf16_copy: bool = False, device_fill_others: bool = False):
    """Step the CUDA path and the oracle side by side; returns {step: worst-error dict}.

    ``oracle_idx``: run the oracle on these tensors only (tensors are independent, so each is
    an exact element-by-element check of the full-size GPU run); None = all tensors.
    ``device_fill_others``: the gradients of the tensors the oracle does NOT follow are drawn on
    the device (same distribution, other bits) instead of on the host; the followed tensors
    always get the host-generated bits the oracle sees.  The next step's host gradients are
    drawn on a background thread while the current step is stepped and compared.
    """
    from concurrent.futures import ThreadPoolExecutor
    hp = dict(w.hparams if hparams is None else hparams)
    n_t = len(w.tensors)
    sel = list(range(n_t)) if oracle_idx is None else list(oracle_idx)
    host_idx = sel if (device_fill_others and oracle_idx is not None) else list(range(n_t))
    gdt = torch.bfloat16 if w.grad_dtype == synth.BF16 else torch.float32
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    hosted = set(host_idx)
    params, dev_p = {}, []
    for i, t in enumerate(w.tensors):
        if i in hosted:
            params[i] = synth.make_param(w, seed, i)
            dev_p.append(torch.from_numpy(params[i]).to(device))
        else:                                        # not followed by the oracle: any values do
            dev_p.append(torch.empty(t.shape, dtype=torch.float32, device=device).normal_(0.0, 0.02, generator=gen))
    pool = ThreadPoolExecutor(max_workers=1)
    draw = lambda step: synth.make_grads(w, seed, step, indices=host_idx, workers=workers)
    pending = pool.submit(draw, 1)
    dev_g = [torch.empty(t.shape, dtype=gdt, device=device) for t in w.tensors]
    opt = binding.CameOptimizer(dev_p, dev_g, flags=flags, bf16_copy=bf16_copy,
                                create_flags=binding.CAME_CREATE_ADAFACTOR if algorithm == "adafactor" else 0)
    no_wd = [bool(flags[i] & binding.CAME_T_NO_WEIGHT_DECAY) for i in sel] if flags else ()
    no_conf = [bool(flags[i] & binding.CAME_T_VEC_NO_CONFIDENCE) for i in sel] if flags else ()
    orc = oracle.OracleOptimizer([params[i] for i in sel], no_weight_decay=no_wd,
                                 vec_no_confidence=no_conf, algorithm=algorithm)
    p0 = [params[i] for i in sel]
    del params
    out = {}
    pos = {i: k for k, i in enumerate(host_idx)}
    for step in range(1, steps + 1):
        grads = pending.result()
        pending = pool.submit(draw, step + 1) if step < steps else None
        for i, dg in enumerate(dev_g):
            if i in hosted:
                dg.copy_(to_torch_grad(torch, grads[pos[i]], device))
            else:
                dg.normal_(0.0, 1e-3, generator=gen)
        opt.step(**hp)
        gs = float(hp.get("grad_scale", 1.0))       # the step's gradient is gs * buffer
        for j, i in enumerate(sel):                  # one tensor at a time keeps the float64 copies small
            g64 = synth.widen(grads[pos[i]])
            orc.step_tensor(j, g64 if gs == 1.0 else g64 * gs, **hp)
        del grads
        if step in check_at:
            torch.cuda.synchronize()
            out[step] = compare_state(opt, orc, None if oracle_idx is None else sel, p0=p0, steps=step)
            if bf16_copy:       # the copy is the kernel's own fp32 result rounded to nearest even
                for p32, p16 in zip(opt.params, opt.p_bf16):
                    want = synth.f32_to_bf16_bits(p32.cpu().numpy())
                    got = p16.view(torch.int16).cpu().numpy().view(np.uint16)
                    assert np.array_equal(got, want), "bf16 parameter copy is not RNE of the fp32 result"
    pool.shutdown()
    opt.close()
    return out
