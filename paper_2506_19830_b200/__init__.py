"""B200-native step-parallel verification pass of Lookahead Reasoning.

The product is the C-ABI library ``liblr_verify.so`` (see ``include/lr_verify.h``);
this package is its thin Python binding plus the in-tree build step.
"""
from .build import build_library, LIB_PATH  # noqa: F401
