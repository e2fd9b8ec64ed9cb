"""PQ-HSA decode-step attention for NVIDIA B200 (sm_100a).

``pqhsa``          thin ctypes binding of the C-ABI library (argument marshalling only)
``workload``       seeded synthetic inputs shaped like the paper's decode workloads
``index_builder``  seeded IVF-PQ index construction (input preparation, not hot path)
"""
