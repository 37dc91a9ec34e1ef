"""Logit post-processing of one row (oracle; test infrastructure).

App. B "Models" fixes only the values: classifier-free guidance scale 3.0,
temperature 1.0, top-k sampling.  The order used here is
guidance -> temperature -> top-k truncation -> softmax, applied in the same way
to the target rows (giving q) and to the drafter rows (giving p).

The pre-softmax value z is defined in float32 so that the top-k threshold is an
exact statement about bit patterns:
    z_j = fl32( fl32(g * (c_j - u_j) + u_j, one rounding) * fl32(1 / tau) )
and without guidance z_j = fl32(l_j * fl32(1 / tau)).  The softmax itself is
evaluated in double precision.
"""

import numpy as np


def fma_f32(a, b, c):
    """Correctly rounded float32 fused multiply-add a*b + c (one rounding).

    a*b is exact in double (48-bit product).  The double sum is then rounded
    to odd using the exact error of the addition, which makes the final
    rounding to float32 equal to a single rounding of the exact value.
    """
    a = np.asarray(a, dtype=np.float32).astype(np.float64)
    b = np.asarray(b, dtype=np.float32).astype(np.float64)
    c = np.asarray(c, dtype=np.float32).astype(np.float64)
    t = np.atleast_1d(a * b)        # exact
    c1 = np.broadcast_to(np.atleast_1d(c), t.shape)
    s = t + c1                      # rounded to double
    bb = s - t                      # exact error of the sum (Knuth two-sum)
    err = (t - (s - bb)) + (c1 - bb)
    even = (s.view(np.int64) & 1) == 0
    toward = np.where(err > 0, np.inf, -np.inf)
    adj = (err != 0) & even & np.isfinite(s)
    s_odd = np.where(adj, np.nextafter(s, toward), s)
    return s_odd.astype(np.float32).reshape(np.shape(a * b + c))


def combine_f32(cond, uncond, cfg_scale, temperature):
    """float32 pre-softmax values z of one row (guidance, then 1/tau)."""
    inv_tau = np.float32(1.0) / np.float32(temperature)
    cond = np.asarray(cond, dtype=np.float32)
    if uncond is None:
        return (cond * inv_tau).astype(np.float32)
    uncond = np.asarray(uncond, dtype=np.float32)
    diff = (cond - uncond).astype(np.float32)
    mixed = fma_f32(np.float32(cfg_scale), diff, uncond)
    return (mixed * inv_tau).astype(np.float32)


def postprocess_row(cond, uncond, cfg_scale, temperature, top_k, allowed_begin=0, allowed_end=None):
    """Return (P, z): the double-precision distribution of one row and its
    float32 pre-softmax values after masking and truncation.

    Tokens outside [allowed_begin, allowed_end) get -inf.  If 0 < top_k < number
    of finite entries, theta is the top_k-th largest z and every z_j < theta
    becomes -inf (all entries equal to theta are kept).
    """
    z = combine_f32(cond, uncond, cfg_scale, temperature).copy()
    V = z.shape[0]
    if allowed_end is None:
        allowed_end = V
    z[:allowed_begin] = -np.inf
    z[allowed_end:] = -np.inf
    finite = np.isfinite(z)
    n_finite = int(finite.sum())
    if top_k > 0 and top_k < n_finite:
        theta = np.sort(z[finite])[n_finite - top_k]
        z[z < theta] = -np.inf
    zd = z.astype(np.float64)
    e = np.exp(zd - zd.max())
    return e / e.sum(), z
