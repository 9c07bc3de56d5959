"""CPU oracle for the EFCP / Sparse M-FAC step (test infrastructure only).

Nothing in the product package may import this.  See efcp_oracle.cpp for what
each routine follows in the paper.
"""
