"""paper_2609_03905_b200: join-agg execution over tensor relations on one B200.

`binding` mirrors the C ABI of libja (include/ja.h); `relations` adds handle/payload conveniences.
"""
from . import binding  # noqa: F401  (raises if libja.so is absent and cannot be built)
from .binding import *  # noqa: F401,F403
from .relations import (Relation, Spec, attention_combine, equal_splits, from_dense, partial_relation, repartition,  # noqa: F401
                        repartition_agg, to_dense)
from .planned_block import PlannedBlock, block_graph, plan_repartition_charges  # noqa: F401,E402
