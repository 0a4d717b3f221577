"""B200 (sm_100a) implementation of the RPTQ hot path (arXiv 2304.01089).

    workloads    seeded synthetic OPT-shaped inputs (no arithmetic of the method)
    calibration  host-side calibration: channel ranges, K-Means, reorder index, Min-Max parameters
    binding      ctypes face of librptq.so (the CUDA kernels behind include/rptq.h)
    shard        token split and max-over-ranks timing for one-process-per-GPU runs
    build        compiles csrc/*.cu into librptq.so with nvcc for sm_100a

`binding` raises ImportError when librptq.so has not been built; nothing falls back to the CPU.
"""
__all__ = ["workloads", "calibration", "binding", "build", "shard"]
