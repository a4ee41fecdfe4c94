"""CPU oracle (test infrastructure only).

`oracle.cnn`  : ctypes wrapper of the plain-C CNN forward/backward and Philox.
`oracle.ps`   : numpy parameter-server state machine (sync / async / replay,
                version ring, checkpoint rollback, chain mirror).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import
this package.  It imports nothing from the CUDA package.
"""
