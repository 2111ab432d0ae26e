"""CPU oracle for ST^3 decode-step attention with visual-token trimming.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this
directory; it exists so that the CUDA path can be checked against a plain,
slow, fp64 restatement of the paper's method.
"""
