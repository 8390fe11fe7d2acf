"""B200-native GVote compression pass (adaptive KV-cache compression by Monte-Carlo voting).

`paper_2509_03136_b200.gvote` is the Python face of the C-ABI library (`include/gvote.h`);
`paper_2509_03136_b200.synth` makes the seeded synthetic workloads.  Importing the package
does not load the CUDA library; the first call into `gvote` does, and fails loudly when the
library has not been built.
"""

__all__ = ["gvote", "synth", "build"]
