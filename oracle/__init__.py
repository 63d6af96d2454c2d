"""CPU oracle for ChunkKV compression: test infrastructure only.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package. The library and its Python binding never do.
"""
