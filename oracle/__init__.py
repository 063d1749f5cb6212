"""TEST INFRASTRUCTURE — fp64 CPU oracle for paged chunked-prefill attention.

Only the tests, ``__graft_entry__.smoke()`` and the CPU-baseline legs of
``bench.py`` may import this package.  It shares no code with the CUDA
library and never imports it.

``reference``  : ctypes wrapper around the plain C implementation (wpp_oracle.c).
``brute``      : separate numpy matrix-form implementation used to pin the C one.
``waves``      : the wave-budget planner and FCFS packing of Section 4.5 (plain Python); some rules the paper
                 leaves open are readings: parity unpinned for those (listed in the module).
``hints``      : chained block hash and gallop/bisect index probe of Section 4.3 (plain Python); the hash function
                 is a reading: parity unpinned for that choice.
``kda``        : the recurrent-state (KDA) update of Section 3.1 token by token in fp64, with the snapshots of
                 Section 3.2 (plain numpy); pinned by a hand-worked example, closed forms and a library solve.
"""
from .reference import (  # noqa: F401
    build,
    oracle_threads,
    oracle_append,
    oracle_attention,
    oracle_attention_units,
    merge_partials,
)
from .brute import brute_dense, gather_contiguous  # noqa: F401
