"""Helpers of the GPU-vs-oracle parity tests: host conversion, oracle driver, tolerance checks.

Tolerances (from the stated targets, see the design notes):
  mask        bit-exact, except rows with |D_oracle - delta| <= 1e-6 or |log pi(a) - log mu(a)| <= 1e-6
  divergence  |gpu - oracle| <= 1e-5 (infinities must coincide)
  loss        relative error <= 1e-4 for fp32 logits, <= 1e-3 for bf16 logits
  dlogits     fp32 output: |gpu - oracle| <= 2e-3 * max|dlogits|;
              bf16 output: |gpu - RN_bf16(oracle)| <= 1 bf16 ulp of the oracle value, and
                           |gpu - oracle| <= (2^-8 + 1e-4) * max|dlogits| (rounding to bf16 alone can
                           exceed 2e-3 * max on the largest elements; the fraction inside the literal
                           2e-3 * max is returned)
"""
import numpy as np
import torch

from oracle import dppo_oracle as O

MASK_BAND = 1e-6
D_TOL = 1e-5


def rows_f64(t, rows=None):
    """Host float64 copy of (selected rows of) a tensor; bf16 / fp32 upcast exactly."""
    if rows is not None:
        t = t[torch.as_tensor(rows, device=t.device, dtype=torch.long)]
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def host_inputs(batch, rows=None):
    sel = (lambda x: None) if False else None
    def pick(x, conv):
        if x is None:
            return None
        if rows is not None:
            x = x[torch.as_tensor(rows, device=x.device, dtype=torch.long)]
        return conv(x.detach().cpu())
    return dict(
        logits=None if batch.logits is None else rows_f64(batch.logits, rows),
        sampled_ids=pick(batch.sampled_ids, lambda x: x.numpy().astype(np.int64)),
        mu_logp=pick(batch.mu_logp, lambda x: x.numpy().astype(np.float64)),
        advantages=pick(batch.advantages, lambda x: x.numpy().astype(np.float64)),
        token_mask=pick(batch.token_mask, lambda x: x.numpy()),
        mu_topk_ids=pick(batch.mu_topk_ids, lambda x: x.numpy().astype(np.int64)),
        mu_topk_p=pick(batch.mu_topk_p, lambda x: x.numpy().astype(np.float64)),
    )


def run_oracle(h, variant, K, delta, scale, want_grad=True, is_cap=None, eps_low=None, given_D=None):
    return O.dppo_loss_fwd_bwd(h["logits"], h["sampled_ids"], h["mu_logp"], h["advantages"], h["token_mask"],
                               variant, K, delta, scale, h["mu_topk_ids"], h["mu_topk_p"], want_grad, is_cap, eps_low, given_D)


def bf16_round(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)


def bf16_ulp(x):
    ax = np.maximum(np.abs(np.asarray(x, dtype=np.float64)), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def check_scalars(gpu_D, gpu_M, ora, h, delta, variant_is_topk=False, eps_low=None):
    """Mask / divergence parity on the rows of `ora`.  Returns the number of exempted rows."""
    gpu_D = np.asarray(gpu_D, dtype=np.float64)
    gpu_M = np.asarray(gpu_M)
    oD, oM = ora["D"], ora["M"]
    fin = np.isfinite(oD)
    assert np.array_equal(np.isfinite(gpu_D), fin), "infinite divergences differ"
    err = np.abs(gpu_D[fin] - oD[fin])
    assert err.size == 0 or err.max() <= D_TOL, f"divergence abs err {err.max():.3e} > {D_TOL}"
    diff = gpu_M != oM
    # exemption bands: D within 1e-6 of delta, or the r >< 1 decision within 1e-6 in the log domain
    valid = np.ones_like(oM, dtype=bool) if h["token_mask"] is None else (h["token_mask"] != 0)
    log_r = np.log(np.where(ora["r"] > 0, ora["r"], 1.0))
    exempt = valid & ((np.abs(oD - delta) <= MASK_BAND) | (np.abs(log_r) <= MASK_BAND))
    if eps_low is not None:
        exempt |= valid & (np.abs(oD - eps_low) <= MASK_BAND)
    bad = diff & ~exempt
    assert not bad.any(), f"mask differs on rows {np.nonzero(bad)[0][:10]} (D={oD[bad][:5]}, delta={delta})"
    return int(exempt.sum()), float(err.max() if err.size else 0.0)


def check_loss(gpu_loss, ora_loss, bf16_inputs, row_loss=None):
    tol = 1e-3 if bf16_inputs else 1e-4
    denom = abs(ora_loss)
    rel = abs(gpu_loss - ora_loss) / denom if denom > 0 else abs(gpu_loss)
    info = dict(rel=rel)
    if row_loss is not None and denom > 0:
        info["kappa"] = float(np.sum(np.abs(row_loss)) / denom)
    assert rel <= tol, f"loss rel err {rel:.3e} > {tol} (gpu {gpu_loss}, oracle {ora_loss}, {info})"
    return info


def check_dlogits(gpu_dl, ora_dl, out_is_bf16, max_abs=None):
    g = gpu_dl.detach().to(torch.float32).cpu().numpy().astype(np.float64)
    o = np.asarray(ora_dl, dtype=np.float64)
    mx = float(np.max(np.abs(o))) if max_abs is None else float(max_abs)
    err = np.abs(g - o)
    if not out_is_bf16:
        assert err.max() <= 2e-3 * mx + 1e-30, f"dlogits err {err.max():.3e} > 2e-3*max ({mx:.3e})"
        return dict(max_err_over_max=float(err.max() / mx) if mx > 0 else 0.0, frac_literal=1.0)
    ulp_err = np.abs(g - bf16_round(o)) / bf16_ulp(o)
    tiny = np.abs(o) < 1e-36          # flushed / subnormal range
    assert np.all((ulp_err <= 1.0) | tiny), f"bf16 dlogits off by {ulp_err[~tiny].max():.2f} ulp"
    assert np.all(np.abs(g[tiny]) < 1e-35)
    assert err.max() <= (2.0 ** -8 + 1e-4) * mx + 1e-30
    frac = float(np.mean(err <= 2e-3 * mx)) if mx > 0 else 1.0
    return dict(max_err_over_max=float(err.max() / mx) if mx > 0 else 0.0, frac_literal=frac,
                max_ulp=float(ulp_err[~tiny].max()) if (~tiny).any() else 0.0)
