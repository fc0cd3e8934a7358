"""fp64 CPU oracle for the token-reduced hybrid prefill.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this
package; the product path never does.  See ``reference.py`` for the definitions.
"""
from .reference import *  # noqa: F401,F403
from .reference import _identity  # noqa: F401
