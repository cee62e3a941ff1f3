"""fp64 CPU oracle (test infrastructure; the product never imports this package)."""
from .ref import (build, phi, ref_backward, ref_backward_mixed, ref_linear, ref_mix, ref_quadratic, ref_relu_backward,  # noqa: F401
                  ref_relu_linear, ref_relu_quadratic, ref_softmax, threads)
