"""CPU oracle of the rollout method (test infrastructure only).

`rollout_theory` holds the paper's graph definitions in pure Python,
`frame_update` binds the plain C implementation of the frame update.  Only
tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do.
"""
