"""Helpers for the tests: golden-file parsing and dense <-> CSR conversion (no op arithmetic)."""
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    """Parse a golden text file: '#' comments, 'key v v v ...' lines, and a 'dense' block."""
    out, dense = {}, None
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tok = line.split()
            if tok[0] == "dense":
                dense = []
                continue
            if dense is not None and len(dense) < out.get("M", 0):
                dense.append([0.0 if t == "." else float(t) for t in tok])
                if len(dense) == out["M"]:
                    out["dense"] = np.array(dense)
                continue
            vals = [float(t) for t in tok[1:]]
            out[tok[0]] = int(vals[0]) if tok[0] in ("M", "K") else np.array(vals)
    return out


def dense_to_csr(dense):
    dense = np.asarray(dense)
    M = dense.shape[0]
    row_ptr = np.zeros(M + 1, dtype=np.int32)
    cols, vals = [], []
    for i in range(M):
        nz = np.nonzero(dense[i])[0]
        cols.extend(nz.tolist())
        vals.extend(dense[i, nz].tolist())
        row_ptr[i + 1] = len(cols)
    return row_ptr, np.array(cols, dtype=np.int32), np.array(vals, dtype=np.float32)


def csr_to_dense(M, K, row_ptr, col_idx, values, dtype=np.float64):
    """Duplicates accumulate."""
    S = np.zeros((M, K), dtype=dtype)
    rows = np.repeat(np.arange(M), np.diff(row_ptr))
    np.add.at(S, (rows, col_idx), values.astype(dtype))
    return S


def csr_rows(row_ptr):
    return np.repeat(np.arange(len(row_ptr) - 1), np.diff(row_ptr))
