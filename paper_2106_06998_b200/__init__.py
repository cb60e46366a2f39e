"""libxconv: XConv activation sketch and randomized-trace weight-gradient estimator on sm_100a.

The CUDA library is loaded on first use of ``paper_2106_06998_b200.binding``; importing the
package alone (for the seeded input generators) touches no native code.
"""
