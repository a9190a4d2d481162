"""B200-native bounded-enumeration repair of sketch holes (the search step of the paper's
symbolic code repair, Section 4.4 / Algorithm 3).  The work is done by the CUDA library
``libxpiler_repair.so`` (C ABI in ``include/xp.h``); this package is its ctypes binding."""
from . import binding  # noqa: F401
from .binding import (EXPORTS, xp_behaviours, marshal_sketches, marshal_grammar, GrammarDesc, summaries_as_numpy, XP_FLAG_ALWAYS_FILTER, XP_FLAG_NO_FILTER, Grammar, HoleResult, LoadedSketch, XpError, load,  # noqa: F401
                      xp_grammar_count, xp_grammar_create, xp_grammar_unrank, xp_int32_peak, xp_int_div_rate, xp_repair,
                      xp_repair_batch, xp_repair_joint, xp_repair_pair, xp_repair_static, xp_result_get, xp_sketch_info_get, xp_sketch_load, xp_sketch_load_batch,
                      xp_sketch_refine, xp_workspace_bytes)
