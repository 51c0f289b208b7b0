"""Structured tensor algebra on densely packed layouts for NVIDIA B200 (sm_100a).

The product is ``libdastac.so`` (C ABI, see ``include/dastac.h``); this package is its Python
binding.  Importing it requires the built library: ``python -m paper_2407_13726_b200.build``.
"""
from .binding import *  # noqa: F401,F403
from .binding import (DastacError, Structure, contract, contract_workspace, launch_count, pack,
                      rank, rank_batch, status_string, structure_count, structure_create, unpack,
                      unrank, unrank_batch)
