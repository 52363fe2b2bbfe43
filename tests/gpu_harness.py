"""Helpers shared by the GPU tests: device-side step buffers and the attention tolerance."""
import numpy as np

from paper_2402_11809_b200.device import DeviceStep, bf16_to_bits, make_context, to_dev  # noqa: F401


def attn_tolerance(ref):
    """Bound on max |err| for one sequence's output: 2e-2 absolute and 1e-2 of the
    RMS of the oracle output.  The RMS is taken per sequence: the sequences of a
    ragged batch are independent problems whose output scale falls as
    1/sqrt(number of keys), so one RMS over the batch would judge short sequences
    by the scale of long ones."""
    rms = float(np.sqrt(np.mean(np.square(ref))))
    return min(2e-2, 1e-2 * rms), rms


def check_attention(got, ref, what=""):
    """got, ref [B, ...]: every sequence within its own tolerance.  Returns the
    largest max|err| / RMS over the sequences."""
    assert np.isfinite(got).all(), what
    worst = 0.0
    for b in range(ref.shape[0]):
        tol, rms = attn_tolerance(ref[b])
        err = float(np.max(np.abs(got[b] - ref[b])))
        assert err <= tol, f"{what} sequence {b}: max|err| {err:.3e} > {tol:.3e} (rms {rms:.3e})"
        worst = max(worst, err / rms)
    return worst
