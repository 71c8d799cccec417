"""Graph descriptors and seeded synthetic inputs shared by the tests, the benchmark,
the CUDA binding and the CPU oracle.  Holds no operator arithmetic."""
from . import descriptor, configs  # noqa: F401
