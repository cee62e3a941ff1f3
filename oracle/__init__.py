"""fp64 CPU oracle (test infrastructure; the product never imports this package)."""
from .ref import build, phi, ref_linear, ref_quadratic, threads  # noqa: F401
