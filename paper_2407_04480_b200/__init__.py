"""B200-native LoCo hot path (arXiv 2407.04480): CUDA library binding and synthetic inputs.

Importing the package loads nothing native; `paper_2407_04480_b200.loco` loads the CUDA
library on first use and raises if it is missing.
"""
