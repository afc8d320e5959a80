"""B200 (sm_100a) implementation of the ANPD draft-and-verify step.

`binding` exposes the C entry points of libanpd_b200.so under their own names;
`build.build()` compiles the library in-tree.  Importing this package does not
load the library; the first call does, and fails loudly if it is missing.
"""
from . import binding, build  # noqa: F401

__all__ = ["binding", "build"]
