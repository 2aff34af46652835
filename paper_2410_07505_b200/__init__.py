"""CrossQuant activation cross-quantizer for NVIDIA B200 (sm_100a).

``paper_2410_07505_b200.cq`` is the binding of the C-ABI library (CUDA kernels);
``paper_2410_07505_b200.workloads`` holds the seeded synthetic inputs.  Importing the
package loads nothing; the CUDA library is loaded on first use of ``cq`` and a missing
library is an error, never a fallback.
"""
__version__ = "0.1.0"
