"""B200-native evaluator of the weight-stationary matrix-multiply recurrence.

``paper_2511_09987_b200.inputs`` makes seeded operands; the CUDA library and its
binding are loaded on first use of :func:`recurrence_matmul` and friends.
"""
__all__ = ["inputs", "binding"]


def __getattr__(name):
    if name in ("binding", "inputs"):
        import importlib
        return importlib.import_module(__name__ + "." + name)
    raise AttributeError(name)
