"""Opt-GQA on B200: paged grouped-query ALiBi attention as a C-ABI CUDA library (sm_100a).

``paper_2505_02351_b200.binding`` is the thin ctypes layer over ``libopt_gqa.so``;
``paper_2505_02351_b200.workloads`` draws the seeded synthetic inputs.
"""
