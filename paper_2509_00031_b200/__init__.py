"""B200-native ZeroQAT hot path: the forward-only two-point zeroth-order QAT step
as hand-written CUDA for sm_100a behind a C-ABI library (see include/zoqat.h).

``binding`` loads the library (and raises if it has not been built); ``synth``
draws the seeded synthetic inputs.  Importing the package loads neither.
"""
