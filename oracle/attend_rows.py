"""Oracle (test infrastructure, not part of the product path): single-query softmax attention over given rows,
the definition written out in numpy fp64.  out[h] = softmax(scale * q[h] . keys[h]^T) . values[h]; this is the
readout equation of Section 3.2 "Readout" for one query whose key / value rows (state readout rows followed
by window tokens, temperatures already folded into `scale`) are handed in.  Only tests/ may import it."""
import numpy as np


def attend_rows(q, keys, values, scale):
    """q [H, d], keys / values [H, n, d] (any float dtype) -> [H, d] float64."""
    q = np.asarray(q, dtype=np.float64)
    keys = np.asarray(keys, dtype=np.float64)
    values = np.asarray(values, dtype=np.float64)
    logits = scale * np.einsum("hd,hnd->hn", q, keys)
    logits -= logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p /= p.sum(axis=1, keepdims=True)
    return np.einsum("hn,hnd->hd", p, values)
