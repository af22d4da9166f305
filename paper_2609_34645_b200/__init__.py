"""B200-native EMU reshard (Nereus plan transitions): a C-ABI CUDA library plus a thin ctypes binding.

``paper_2609_34645_b200.binding``  the binding; importing it loads the CUDA library and fails loudly when it
                                  has not been built.
``paper_2609_34645_b200.inputs``   seeded synthetic inputs and the benchmark configurations (no reshard
                                  arithmetic).
"""
