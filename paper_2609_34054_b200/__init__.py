"""B200-native shared-base + low-rank KV-cache path (PReCache hot path).

``inputs``  seeded synthetic workloads (no GPU needed)
``binding`` thin ctypes layer over the C-ABI library ``libprecc.so`` (loaded lazily;
            every call fails loudly if the library is missing -- there is no fallback)
"""
