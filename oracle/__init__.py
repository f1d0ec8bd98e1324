"""CPU oracle for the ZeroQuant-HERO W8A8 transformer-layer forward.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain, fp64 / exact-integer
statement of what the quantized layer computes, written from the paper's
equations (Sec. 2.1-2.3).  It shares no code with the CUDA library and never
imports it.  Only the tests, the smoke check and the benchmark's CPU-baseline
leg may import it; the product path never does.

Modules
-------
quant   Sec. 2.1 quantizers (symmetric INT8, column-wise weights, TWQ/FWQ/SQ)
ops     the quantization-aware operators (LN^quant, GeMM^quant, attention, GELU^quant)
layer   offline preparation (calibration, Eq. 20-23/32 folding) and the
        layer forward of Sec. 2.2 under the module modes of Table 1
search  per-module sensitivity and the greedy INT8 -> FP mode search that
        generalises Table 1's presets (Sec. 2.3), as loops over `layer`

Pins (what fixes each function to something other than itself) live in
tests/test_oracle_*.py.  The whole INT8 layer has no external definition to
the last bit; it is pinned in two ways: every rounding decision piecewise
(integer contractions, quantizers, folding identities, LayerNorm / GELU /
softmax closed forms, the all-FP layer against a library transformer layer),
and the wiring of the layer stage by stage: each operator of layer_forward,
in every mode of Table 1, against the float64 library routine of that operator
fed the dequantized border the oracle itself fed it, to within the operator's
quantization steps, plus a bound against the unquantized layer end to end.
"""
