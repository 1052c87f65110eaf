"""Float64 CPU oracle of the MI hook (test infrastructure; never on the product path)."""
from .mi_hook import *   # noqa: F401,F403
