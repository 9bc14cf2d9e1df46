"""fp64 CPU oracle of the optimiser step that follows the block's backward pass: global-norm gradient clipping over all
gradient tensors, then SGD with Nesterov momentum and per-group learning rate / weight decay.

TEST INFRASTRUCTURE ONLY (same rules as the rest of this package: only tests, the smoke check and the benchmark's CPU
legs may import it; it shares nothing with the CUDA library).

The paper (Sec. 3.2 "Optimization"; Table 1 "Optimization"; Table 2 rows 6-7) names the method -- SGD, Nesterov momentum
0.937, three parameter groups (decayed weights, undecayed normalisation gains, undecayed biases), global-norm clip 10.0
every step computed as ONE squared-norm accumulation over all 243 gradient tensors -- and says it carries the dominant
framework's default semantics, without printing formulas.  Those defaults, written out:

  clip:   total = sqrt(sum over every tensor and element of g^2);  c = max_norm / (total + 1e-6);  g <- g * min(c, 1)
  update: d   = g + weight_decay * p
          buf = d                      on the first step (no momentum buffer yet)
          buf = momentum * buf + d     afterwards (dampening 0)
          p  <- p - lr * (d + momentum * buf)          (Nesterov form)

Pins (tests/test_oracle_pins_optimizer.py): hand-worked numbers, the framework's own CPU optimiser and clipping routine
in float64 over several steps and groups, no-op clipping below the threshold, exact norm after clipping, momentum 0
reducing to plain gradient descent.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np


def global_norm(grads) -> float:
    """sqrt of the sum of squares over every element of every tensor (one accumulation, fp64)."""
    total = 0.0
    for g in grads:
        g = np.asarray(g, dtype=np.float64)
        total += float((g * g).sum())
    return float(np.sqrt(total))


def clip_coefficient(total_norm: float, max_norm: float) -> float:
    return min(float(max_norm) / (float(total_norm) + 1e-6), 1.0)


def clip_global_norm(grads, max_norm: float):
    """Returns (clipped gradients as new fp64 arrays, total norm before clipping)."""
    total = global_norm(grads)
    c = clip_coefficient(total, max_norm)
    return [np.asarray(g, dtype=np.float64) * c for g in grads], total


def sgd_nesterov_update(p, g, buf, lr: float, momentum: float, weight_decay: float, first_step: bool):
    """One tensor: returns (new parameter, new momentum buffer) as fp64 arrays; g is the (already clipped) gradient."""
    p = np.asarray(p, dtype=np.float64)
    d = np.asarray(g, dtype=np.float64) + float(weight_decay) * p
    new_buf = d.copy() if first_step else float(momentum) * np.asarray(buf, dtype=np.float64) + d
    step = d + float(momentum) * new_buf
    return p - float(lr) * step, new_buf


def clip_sgd_step(params, grads, bufs, groups, lr, weight_decay, momentum: float, max_norm: float, first_step: bool):
    """The whole step over a list of tensors.  groups[i] in {0, 1, 2} selects lr[group], weight_decay[group].
    Returns (new params, new buffers, total gradient norm before clipping)."""
    clipped, total = clip_global_norm(grads, max_norm)
    new_p, new_b = [], []
    for p, g, b, grp in zip(params, clipped, bufs, groups):
        q, nb_ = sgd_nesterov_update(p, g, b, lr[grp], momentum, weight_decay[grp], first_step)
        new_p.append(q)
        new_b.append(nb_)
    return new_p, new_b, total


# ------------------------------------------------------------------ dynamic loss scaling (Sec. 3.2 "Mixed precision", Table 1, Table 2 row 4)
def scaled_clip_sgd_step(params, grads, bufs, groups, lr, weight_decay, momentum: float, max_norm: float, first_step: bool,
                         scale: float, growth_tracker: int, growth_factor: float = 2.0, backoff_factor: float = 0.5,
                         growth_interval: int = 2000, floor: float = 0.0):
    """One optimiser step when the gradients arrive multiplied by the loss scale (the paper's recipe: initial scale 2^16,
    dynamic, with a FLOOR -- Table 2 row 4: without it per-rank overflows drove the scale towards zero).  The dominant
    framework's scaler semantics, which the paper keeps:

      unscale: g <- g / scale;  if any gradient element is inf or NaN the step is SKIPPED (parameters and momentum
      untouched), scale <- max(scale * backoff_factor, floor), growth_tracker <- 0;
      otherwise clip + update as clip_sgd_step on the unscaled gradients, growth_tracker += 1, and after growth_interval
      consecutive good steps scale <- scale * growth_factor, growth_tracker <- 0.

    Returns (params, bufs, total_norm of the unscaled gradients or inf/nan, scale, growth_tracker, skipped)."""
    inv = 1.0 / float(scale)
    unscaled = [np.asarray(g, dtype=np.float64) * inv for g in grads]
    finite = all(bool(np.isfinite(g).all()) for g in unscaled)
    if not finite:
        return list(params), list(bufs), float("nan"), max(float(scale) * backoff_factor, float(floor)), 0, True
    new_p, new_b, total = clip_sgd_step(params, unscaled, bufs, groups, lr, weight_decay, momentum, max_norm, first_step)
    growth_tracker += 1
    if growth_tracker == growth_interval:
        scale, growth_tracker = float(scale) * growth_factor, 0
    return new_p, new_b, total, float(scale), growth_tracker, False
