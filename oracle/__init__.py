"""CPU oracle for the cold-start convolution path.

TEST INFRASTRUCTURE ONLY.  Slow, plain, fp64 restatements of what the CUDA
path computes, written from the paper and the textbook definitions it relies
on.  Only tests/, the smoke check and the benchmark's CPU-baseline leg may
import this package; the product package never does, and this package never
imports the product.

Parity pins (tests/test_oracle_*.py, all CPU):
  winograd.matrices_exact  exact-rational 1-D correlation identity on all basis pairs
  winograd.filter_transform  pseudo-inverse round trip; plane count / byte ratio of the
                             paper's Figure 3 / Table 2; closed-form transform of
                             centre-tap and all-ones filters
  winograd.winograd_conv   equals conv.direct_conv on ragged sizes (pins tiling/edges)
  conv.direct_conv         1x1 conv == matmul; depthwise == per-channel correlation;
                           delta filters == shifts; library conv2d in fp64 on CPU;
                           pure-Python loop version on tiny shapes
  pack.pack_weights        brute-force bijection + zero padding on tiny shapes;
                           bf16 rounding against hand-computed bit patterns
  selection.*              the paper's Table 2 worked example; brute-force enumeration
                           on random small integer tables
  conv.maxpool/gavgpool    closed forms on ramps / constants
  scheduler.simulate       hand-computed makespans; an independent unit-time tick simulator
                           on random layer graphs
  scheduler.schedule/search  hand examples; fixed point of the balancing loop; bounded by
                           brute force over all queue assignments and by queue 0's own load;
                           exhaustive search no worse than any single combination
"""
