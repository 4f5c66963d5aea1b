"""B200 (sm_100a) Virtual-Expert MoE-layer forward of SwapMoE behind a C ABI.

``inputs``  - seeded synthetic workloads (no method arithmetic);
``binding`` - ctypes handle on libswapmoe.so (loaded lazily, built in-tree);
``build``   - nvcc build of the library.
"""
