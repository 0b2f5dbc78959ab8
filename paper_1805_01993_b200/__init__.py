"""Compressed coded distributed computing shuffle for one B200.

``paper_1805_01993_b200.inputs``  seeded synthetic inputs (no method arithmetic)
``paper_1805_01993_b200.ccdc``    Python binding of the C-ABI CUDA library

Importing the package loads nothing; ``ccdc`` loads the shared library on first
use and raises if it has not been built.
"""
