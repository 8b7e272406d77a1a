"""B200 (sm_100a) Tune-mode Convolution-BatchNorm: C-ABI CUDA library and its thin binding.

``inputs`` (synthetic data, layer shapes) imports without the compiled library; the binding
(``convbn``) loads ``libconvbn.so`` on first use and raises if it is missing.
"""
