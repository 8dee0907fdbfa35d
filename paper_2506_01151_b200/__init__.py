"""B200-native vocabulary masking for grammar-constrained decoding (ZapFormat / Formatron).

The work is done by the CUDA library built from csrc/ (C-ABI in include/fmt.h); this package
is its thin Python binding.
"""
from ._build import build  # noqa: F401
from .binding import (  # noqa: F401
    BF16, FP32, FMT_OK, ERR_CAPACITY, ERR_FINISHED, ERR_INVALID_ARG, ERR_TOKEN_REJECTED, ERR_GRAMMAR_SYNTAX,
    ERR_UNDEFINED_SYMBOL, ERR_EMPTY_LANGUAGE, EXPORTS, NOALLOC_MAX_CHARTS, FmtError, Grammar, State, apply_mask,
    fill_mask_noalloc, json_schema_to_ebnf, lib,
)
