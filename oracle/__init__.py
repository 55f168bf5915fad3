"""CPU oracle for the QZO hot path (test infrastructure, not a product path).

Everything under ``oracle/`` is a plain, slow, obviously-correct restatement of
what the paper's method computes, in fp64 numpy.  It shares no code with the
CUDA library and is imported only by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product path never calls into it.

Modules
-------
philox   counter-based Philox4x32-10, uniforms, Box-Muller normals, z(seed, i)
int4     nibble pack / unpack and the symmetric group quantiser (Eq. 3, Eq. 4)
linear   perturbed de-quantised linear layer (Eq. 4, Eq. 5)
model    Llama-style and OPT-style decoder forward + next-token cross entropy
qzo      one step of Algorithm 1 from the untouched scales (Eq. 5), the in-place
         perturbation it is pinned against, directional-derivative clipping
         (Eq. 6), seeded scale update

Parity status: every function here is pinned by ``tests/test_oracle_*.py``
except the full-model loss values (the paper prints no worked example), which
are marked "parity unpinned" in ``model.py``.
"""
