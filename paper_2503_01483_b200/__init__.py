"""KurTail rotation learning on B200 (sm_100a): ctypes binding over libkurtail.

`kurtail` holds the binding (loaded lazily, so importing this package needs no
GPU), `synth` the seeded input generators, `build` the nvcc build step.
"""
