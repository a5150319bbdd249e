"""qil: B200 (sm_100a) low-bit quantised linear layers behind a C ABI.

``paper_2412_01034_b200.api`` is the thin Python binding (argument marshalling
only; every step runs in the CUDA library ``libqil.so``).  Importing this package
does not load the library; ``api`` does, and raises if it has not been built.
``workloads`` holds the seeded synthetic input generators.
"""

__all__ = ["api", "workloads", "build"]
