"""fp64 CPU oracle for the last-dimension softmax -- test infrastructure only.

Nothing in the product package imports this directory; see ``fso.py``.
"""
