// Process-wide measurement and debugging switches of libbigmac.  The defaults are the product; they change only
// through bigmac_debug_set (bigmac_debug.h).  The library never reads the environment.
#pragma once

namespace bigmac {

struct Switches {
    int overlap = 1;        // backward pass: independent launches on the handle's second stream (0: one stream)
    int tc_pair = 1;        // CTA-pair tcgen05 kernel where it is the faster one (0: one-CTA kernel everywhere)
    int groupk = 1;         // dynamically scheduled per-expert weight-gradient kernel where it pays (0: never)
    int fused_mlp = 1;      // inference: expert GEMM1 + sigma + GEMM2 in one kernel on short tile lists (0: never, 2: always)
    int epi_parts = 0;      // working epilogue warps per lane quadrant of plain epilogues (1, 2, 4; 0: the default, 2)
    int staged_stores = 1;  // wide bf16 outputs leave through shared-memory boxes and TMA stores (0: always 32-byte direct stores)
    int fuse_dispatch = 0;  // 1: expert GEMM1 (and dW1) gather the rows of x' themselves, no dispatch launch, no grouped copy.
                            // Off by default: the gathered operand loads (16-byte asynchronous copies by two extra warps)
                            // feed the mainloop at half the rate of TMA boxes (large workload: expert GEMM1 1.08 ms against
                            // 0.73 + 0.07 ms for the dispatch, dW1 1.20 against 0.47 ms)
    int chain = 1;          // kernels of a call are launched with programmatic stream serialisation: a grid is set up while
                            // its predecessor still runs and waits (griddepcontrol.wait) before it touches memory (0: plain launches)
    unsigned tc_mask = ~0u; // bit i: contraction i runs on tcgen05 (read when a handle is created)
};

Switches& switches();

}  // namespace bigmac
