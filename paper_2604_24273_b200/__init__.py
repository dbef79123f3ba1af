"""BitLinear W1.58A8 hot path of the BitRL frozen backbone, as hand-written CUDA for sm_100a.

``bitrl``  - thin ctypes binding of the C-ABI library (argument marshalling only).
``inputs`` - seeded synthetic input generators (no arithmetic of the method).
"""
__all__ = ["bitrl", "inputs"]
