"""B200 (sm_100a) streaming-scan hot path of S^3-Attention: SAE Top-k encode, CSR postings,
host-resident inverted index, co-activation span scoring. All compute runs in the CUDA library
behind include/s3.h; this package only marshals arguments (see binding.py)."""
from .binding import *  # noqa: F401,F403
