"""B200-native grouped gradient aggregation + parameter update (STAR's
parameter-server hot path) behind a C-ABI CUDA library.

``paper_2512_09685_b200.binding`` loads the library and mirrors its entry
points; ``paper_2512_09685_b200.workloads`` makes the seeded synthetic inputs.
Importing the package itself loads nothing.
"""
