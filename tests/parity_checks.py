"""Finer-grained comparisons for the parity tests.

A whole-tensor rel-L2 lets an error that is confined to a few low-energy outputs hide: with a |k|^-2 field a
retained mode at |k| = 16 carries 1/256 of the energy of one at |k| = 1, and a single wrong plane is 1/N_0 of a
grid tensor.  These checks look at every retained mode and at every plane on its own scale."""
import numpy as np

MODE_TOL = 1e-4     # max error of a mode's entries over the rms of that mode's entries
PLANE_TOL = 1e-5    # rel-L2 of each plane (fixed index along the first grid dimension)
FLOOR = 0.05        # a mode weaker than this share of the tensor's rms is measured against the share instead


def per_mode_excess(got, ref, lead_dims=2):
    """max over modes m of  max_{lead} |got[.., m] - ref[.., m]| / max(rms_{lead} |ref[.., m]|, FLOOR * rms(ref)),
    for spectra shaped [lead..., modes...] (lead = (B, C) or (C_in, C_out)); returned as a multiple of MODE_TOL."""
    got = np.asarray(got).astype(np.complex128)
    ref = np.asarray(ref).astype(np.complex128)
    lead = int(np.prod(ref.shape[:lead_dims]))
    g, r = got.reshape(lead, -1), ref.reshape(lead, -1)
    num = np.abs(g - r).max(axis=0)
    rms_m = np.sqrt(np.mean(np.abs(r) ** 2, axis=0))
    rms_all = float(np.sqrt(np.mean(np.abs(r) ** 2)))
    den = np.maximum(rms_m, FLOOR * rms_all)
    if rms_all == 0.0:
        return float(num.max() > 0.0) * np.inf if num.max() > 0.0 else 0.0
    return float((num / den).max() / MODE_TOL)


def per_plane_excess(got, ref, plane_axis=2):
    """max over the planes along `plane_axis` (and over the leading batch/channel entries) of the plane's
    rel-L2, as a multiple of PLANE_TOL; planes whose reference is weaker than FLOOR of the tensor's rms are
    measured against that share."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.ndim <= plane_axis + 1:            # a 1-D grid has no planes: one "plane" per (b, c) row
        plane_axis = ref.ndim - 2
    n_lead = int(np.prod(ref.shape[:plane_axis + 1]))
    g, r = got.reshape(n_lead, -1), ref.reshape(n_lead, -1)
    err = np.sqrt(np.sum((g - r) ** 2, axis=1))
    nrm = np.sqrt(np.sum(r ** 2, axis=1))
    floor = FLOOR * float(np.sqrt(np.mean(r ** 2))) * np.sqrt(r.shape[1])
    if floor == 0.0:
        return 0.0 if err.max() == 0.0 else np.inf
    return float((err / np.maximum(nrm, floor)).max() / PLANE_TOL)
