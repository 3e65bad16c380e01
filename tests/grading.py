"""Tolerance rules used by the GPU parity tests (the oracle decides; the paper fixes no tolerance).

assign : indices bit-exact, except that a GPU index g != oracle index is excused iff
         d64(x, c_g) - d64(x, c_best) < 1e-3 * (|x|^2 + |c_best|^2); excused near-ties are counted.
dist   : |dist_gpu - d64(x, c_g)| <= 1e-3 * (|x|^2 + |c_g|^2).
update : counts exact; per-centroid |c_gpu - c_oracle|_2 <= 1e-3 * max(|c_oracle|_2, 1e-6 sqrt(D)).
inertia: relative 1e-3.
"""
import numpy as np

from oracle import kmeans_oracle as orc

TIE_TOL = 1e-3
CENTROID_TOL = 1e-3
INERTIA_TOL = 1e-3


def grade_assign(Xb, Cb, idx_gpu, dist_gpu=None, rows=None):
    """Xb [N,D], Cb [K,D] bf16 bits (numpy); idx_gpu/dist_gpu numpy. `rows` restricts to a sample."""
    if rows is not None:
        Xb, idx_gpu = Xb[rows], idx_gpu[rows]
        dist_gpu = None if dist_gpu is None else dist_gpu[rows]
    idx_o, dist_o, _ = orc.assign(Xb, Cb)
    K = Cb.shape[0]
    assert idx_gpu.min() >= 0 and idx_gpu.max() < K, "GPU index out of range"
    X = orc.bf16_to_f64(Xb)
    C = orc.bf16_to_f64(Cb)
    xn = (X * X).sum(1)
    cn = (C * C).sum(1)
    d_g = orc.pair_sqdist(Xb, C, idx_gpu)
    mism = idx_gpu != idx_o
    tau = TIE_TOL * (xn + cn[idx_o])
    unexcused = mism & ~((d_g - dist_o) < tau)
    report = {"n": int(len(idx_o)), "mismatch": int(mism.sum()), "unexcused": int(unexcused.sum()),
              "max_gap_rel": float(((d_g - dist_o) / (xn + cn[idx_o] + 1e-300)).max()) if len(idx_o) else 0.0}
    assert not unexcused.any(), f"assign parity: {report}, first bad rows {np.nonzero(unexcused)[0][:8]}"
    if dist_gpu is not None:
        err = np.abs(dist_gpu.astype(np.float64) - d_g)
        bound = TIE_TOL * (xn + cn[idx_gpu])
        report["max_dist_err_rel"] = float((err / (xn + cn[idx_gpu] + 1e-300)).max()) if len(err) else 0.0
        assert (err <= bound).all(), f"dist parity: {report}"
        assert (dist_gpu >= 0).all()
    return report


def grade_update(Xb, idx, K, C_prev_bits, C_gpu, C_bits_gpu, counts_gpu):
    """Teacher-forced: the oracle updates from the SAME idx the GPU update consumed."""
    C_o, counts_o = orc.update(Xb, idx, K, C_prev_bits)
    assert np.array_equal(counts_gpu.astype(np.int64), counts_o), "counts differ"
    D = Xb.shape[1]
    err = np.linalg.norm(C_gpu.astype(np.float64) - C_o, axis=1)
    bound = CENTROID_TOL * np.maximum(np.linalg.norm(C_o, axis=1), 1e-6 * np.sqrt(D))
    report = {"max_centroid_err_rel": float((err / np.maximum(np.linalg.norm(C_o, axis=1), 1e-30)).max()),
              "empty": int((counts_o == 0).sum())}
    assert (err <= bound).all(), f"centroid parity: {report}"
    empty = counts_o == 0
    if empty.any():   # kept centroids are bit-exact
        prev = orc.bf16_to_f64(C_prev_bits) if C_prev_bits is not None else np.zeros_like(C_o)
        assert np.array_equal(C_gpu[empty].astype(np.float64), prev[empty])
    if C_bits_gpu is not None:  # the bf16 copy is the RNE rounding of the GPU's own fp32 means
        assert np.array_equal(C_bits_gpu, orc.f64_to_bf16(C_gpu.astype(np.float64)))
    return report
