"""CPU oracle for the BiCache attention hot path.

TEST INFRASTRUCTURE ONLY.  This package is the plain, slow, fp64 statement of
what the library must compute.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg, and by nothing else; the
product path never routes through it.  It shares no code with the CUDA path
and imports nothing from it.

Parity status of each function (what pins it, see tests/test_oracle_*.py):

  reuse_depth      pinned (hand-computed cases, ranges, monotonicity).  The
                   *contents* of the depth table are an input; the paper
                   prints no table values, so the stand-in table used by the
                   workloads is "parity unpinned".
  PagedPrefixStore pinned (independent trace simulation, conservation laws).
  attention        pinned (scalar brute force, torch SDPA fp64, closed forms,
                   rational-weight golden cases, invariances).
  merge            pinned (any split of the key set equals the direct result).
  attend/attend_full/stack
                   pinned (brute force over the concatenated key list, depth-0
                   and depth-L special cases, cached == fresh special case).
  is_refresh_step/attend_step (Eq. 5)
                   pinned (refresh steps enumerated by hand for Delta = 16;
                   Delta = 1 equals full recompute at every step; a separate
                   brute force that looks up "the step whose prefix KVs are in
                   use" in closed form and concatenates; prefix KVs constant
                   over the steps make the result independent of Delta).
  kv_similarity/depth_from_similarity/build_depth_table (Eq. 3, Sec. 5.1)
                   pinned (closed forms: identical, negated, scaled and
                   orthogonally mixed tensors with cos = a / sqrt(a^2 + b^2);
                   scalar-loop brute force; hand-written threshold and
                   averaging cases).
  xxh64/prefix_key (Sec. 5.2, k = h(p))
                   pinned (the published digests of the empty input and of "a",
                   and the `xxhash` library on random inputs of every tail length).
  project_kv (Eq. 1)
                   pinned (scalar-loop brute force, selector weights that copy
                   chosen hidden components, linearity).
  rope_rotate      pinned (zero angle, quarter turn, scalar loop, norm of every
                   pair preserved, inner products depend on the position
                   difference only).  The paper names no position encoding: the
                   angles are an input.
"""
from .bicache_oracle import (  # noqa: F401
    OracleError,
    InvalidArgument,
    OutOfPages,
    NotFound,
    reuse_depth,
    PagedPrefixStore,
    attention,
    is_refresh_step,
    attend_step,
    kv_similarity,
    depth_from_similarity,
    build_depth_table,
    xxh64,
    prefix_key,
    project_kv,
    rope_rotate,
    merge,
    attend,
    attend_full,
    attend_rows,
    attend_full_rows,
    stack,
)
