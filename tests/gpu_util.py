"""Test-side re-export of the harness helpers."""
from paper_2609_39813_b200.harness import NormLinearGpu, ceil16, down, rel_l2, up  # noqa: F401
