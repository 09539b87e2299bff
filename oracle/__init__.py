"""TEST INFRASTRUCTURE: CPU eager oracle (see eager_ops.c and eager.py)."""
