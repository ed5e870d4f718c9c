"""PureKV hot path for B200 (sm_100a): ST-SpAttn prefill, low-layer window scores,
budgeted top-h selection and K/V compaction, as a C-ABI CUDA library plus this
thin ctypes binding.  `inputs` (seeded synthetic workloads) imports nothing else
from the package; `binding` loads the compiled library and fails if it is absent."""
__version__ = "0.1.0"
