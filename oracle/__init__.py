"""CPU oracle for LayerPipe's delayed-gradient training step.

TEST INFRASTRUCTURE ONLY.  Everything in this package is a plain, slow,
by-eye-checkable restatement of the paper's equations in numpy.  It exists so
that tests, the smoke check and the benchmark's CPU-baseline leg have something
independent to compare the CUDA library against.  The product path never
imports it, and it never imports the product package.
"""
