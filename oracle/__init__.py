"""CPU oracle for the linear data-movement operators and the two distributed layers.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, deliberately naive
numpy restatement of what the operators compute (broadcast B, sum-reduce R = B*,
halo exchange H, adjoint halo exchange H*, the generalized all-to-all with scatter and
gather as special cases, all-reduce, the broadcast / sum-reduce along partition dimensions, the distributed depthwise convolution, the 3-D star-stencil layer,
the distributed pooling layer and the distributed affine layer, each with its adjoint).  Nothing in the product
package imports it; only the test-suite, the smoke check and the CPU-baseline leg
of the benchmark may call it.  It shares no code, table or helper with the CUDA
path and imports nothing but numpy.

Every function cites the passage of the paper (Hewett & Grady, "A Linear
Algebraic Approach to Model Parallelism in Deep Learning") that it restates.

Pin status: every function here is pinned by the CPU tests against something
other than itself (hand-built operator matrices, values printed in the paper's
Appendix B figures, closed forms, library routines on the unpartitioned tensor).
No function is "parity unpinned".
"""

from .partition import Partition, balanced_split, halo_widths_1d  # noqa: F401
from .primitives import (  # noqa: F401
    broadcast_fwd,
    broadcast_adj,
    sumreduce_fwd,
    sumreduce_adj,
    halo_fwd_definition,
    halo_fwd_sequence,
    halo_adj_sequence,
    adjoint_test_ratio,
    assemble_global,
    scatter_global,
    repartition_fwd,
    repartition_adj,
    allreduce,
    partition_broadcast_fwd,
    partition_broadcast_adj,
    round_to_bf16_bits,
    bf16_add,
)
from .layers import (  # noqa: F401
    conv_fwd,
    conv_adj,
    conv_adj_scatter_then_halo,
    conv_adj_params,
    convg_fwd,
    convg_adj,
    convg_adj_params,
    stencil3d_fwd,
    stencil3d_adj,
    stencil3d_fwd_exchange_then_local,
    affine_fwd,
    affine_adj,
    affine_adj_params,
    bf16_bits_to_f64,
    pool_partition,
    pool_fwd_global,
    pool_adj_global,
    pool_fwd,
    pool_adj,
)
