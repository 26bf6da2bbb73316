"""Small shared helpers for the tests (no arithmetic of the method)."""
import dataclasses

import numpy as np


def batch_dict(batch):
    """DagBatch dataclass -> plain dict with the same field names (what the oracle takes)."""
    return {f.name: getattr(batch, f.name) for f in dataclasses.fields(batch)}


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64)))) if np.size(a) else 0.0
