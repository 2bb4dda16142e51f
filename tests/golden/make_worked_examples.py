"""Writes worked_examples.json: tiny BitLinear examples worked by hand from Eq. 1-7, 11, 12.

Nothing here calls the oracle or the CUDA path; the only arithmetic is the closed-form
gamma = 3.5 / sqrt(5.25) and the two final products, everything else is typed in from the
hand derivation quoted in each entry.
"""
import json
import math
import os

gamma = 3.5 / math.sqrt(5.25)
fx = {
    "binarize_2x8": {
        "citation": "Eq. 1-3 (Sign(W - alpha), Sign(0) = -1, alpha = mean W) and Eq. 12 (beta = mean |W|), worked by hand",
        "derivation": "sum W = 2.0 + 2.0 = 4.0 over 16 entries -> alpha = 0.25; sum |W| = 6.0 + 5.5 = 11.5 -> beta = 0.71875; "
                      "row0 - alpha = [.25,-.75,1.25,-1.75,0,0,.25,.75] -> signs + - + - - - + + -> LSB-first byte 1+4+64+128 = 197; "
                      "row1 - alpha = [-1.25,1.75,0,.25,-.5,.5,0,-.75] -> signs - + - + - + - - -> byte 2+8+32 = 42; "
                      "row0 has 4 plus, 4 minus -> rowsum 0; row1 has 3 plus, 5 minus -> rowsum -2",
        "W": [[0.5, -0.5, 1.5, -1.5, 0.25, 0.25, 0.5, 1.0], [-1.0, 2.0, 0.25, 0.5, -0.25, 0.75, 0.25, -0.5]],
        "alpha": 0.25, "beta": 0.71875, "bytes": [197, 42], "rowsum": [0, -2]},
    "absmax_ties_noLN": {
        "citation": "Eq. 4-5 with Q_b = 128, gamma = max|x| = 128 so the scale is exactly 1; round-half-to-even, clip to +-(Q_b - 1)",
        "derivation": "64->64; -128->-128 clipped to -127; 0.5->0; 1.5->2; 2.5->2; -0.5->0; -1.5->-2; 127.4->127",
        "x": [64.0, -128.0, 0.5, 1.5, 2.5, -0.5, -1.5, 127.4], "gamma": 128.0,
        "codes": [64, -127, 0, 2, 2, 0, -2, 127]},
    "eta_noLN": {
        "citation": "Eq. 6: eta = min x, range scaled into [0, Q_b]; gamma read as max x - min x",
        "derivation": "eta = -2, gamma = 6 - (-2) = 8, scale 16; (x - eta)*16 = 0,32,64,128->127,48,80,16,112",
        "x": [-2.0, 0.0, 2.0, 6.0, 1.0, 3.0, -1.0, 5.0], "eta": -2.0, "gamma": 8.0,
        "codes": [0, 32, 64, 127, 48, 80, 16, 112]},
    "ln_absmax_1to8": {
        "citation": "Eq. 12 LN (population variance, eps = 0) then Eq. 4-5",
        "derivation": "mean 4.5, variance 5.25; xhat = (x-4.5)/sqrt(5.25); gamma = 3.5/sqrt(5.25); "
                      "codes = rne((x-4.5)/3.5*128) = -128->-127, -91.43->-91, -54.86->-55, -18.29->-18, 18, 55, 91, 127",
        "x": [1, 2, 3, 4, 5, 6, 7, 8], "ln_eps": 0.0, "gamma": gamma,
        "codes": [-127, -91, -55, -18, 18, 55, 91, 127]},
    "forward_2x8": {
        "citation": "Eq. 7 and Eq. 11 on the two fixtures above: y = acc * beta * gamma / Q_b",
        "derivation": "row0 signs + - + - - - + +: -127+91-55+18-18-55+91+127 = 72; "
                      "row1 signs - + - + - + - -: 127-91+55-18-18+55-91-127 = -108; y = acc * 0.71875 * (3.5/sqrt(5.25)) / 128",
        "acc": [72, -108], "y": [72 * 0.71875 * gamma / 128, -108 * 0.71875 * gamma / 128]},
}
out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "worked_examples.json")
with open(out, "w") as f:
    json.dump(fx, f, indent=1)
