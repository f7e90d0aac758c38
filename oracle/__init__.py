"""CPU oracle of the NITI integer training ops -- test infrastructure, never a product path.

Only ``tests/``, the smoke check and the bench's CPU-baseline / reference arm import this
package.  It shares no code with the CUDA library and does not import it.
"""
from .ref import *  # noqa: F401,F403
from .net import oracle_train_step, OracleNetState  # noqa: F401
