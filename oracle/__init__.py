"""CPU oracle for streamed-KV verification attention.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this; only
the tests, the smoke check and the benchmark's CPU-baseline leg do.  The code
here is deliberately plain and slow (fp64 numpy, no blocking or fusion) so it
can be checked against the paper by eye, and it shares nothing with the CUDA
path.
"""
from .attention import verify_attention, verify_attention_rows  # noqa: F401
from .streaming import (chunk_partial, merge, streamed_verify_attention,  # noqa: F401
                        IDENTITY)
from .commit import cohort_build, commit_gather, migration_endpoint  # noqa: F401
from .width import WidthController  # noqa: F401
