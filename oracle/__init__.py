"""fp64 CPU oracle for multiquery decode attention (test infrastructure only).

Nothing in the product package imports this; see ``oracle/mqa_ref.c``.
"""
