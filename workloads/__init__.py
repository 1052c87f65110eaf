"""Seeded synthetic inputs for the MI hook (data only; none of the method's arithmetic)."""
from .spec import *          # noqa: F401,F403
from .configs import (BASE_SEED, CONFIG_NAMES, make_chained, make_config, make_decode, make_mixed, make_replay,  # noqa: F401
                      make_sae_heavy, make_sae_weights, make_tiny, ragged_lengths_lognormal,
                      ragged_lengths_uniform, replay_map)
from .install import install, make_context  # noqa: F401,E402
