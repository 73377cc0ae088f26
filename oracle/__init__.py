"""Float64 CPU oracle (test infrastructure only; never on the product path).

`oracle.api` wraps the plain-C definitions in `invconv_oracle.c`;
`oracle.dense` is the even plainer layer for tiny inputs (dense matrix,
Gaussian elimination, the literal recursions of Theorems 1 and 2).
Nothing here imports, or is imported by, the CUDA package.
"""
