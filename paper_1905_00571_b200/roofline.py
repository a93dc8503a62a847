"""Sparse-roofline accounting for a model description (reporting only, no layer arithmetic).

Per layer: t_roof = max(2 * nonzero MACs / R_cuda, (compressed weights + activations
in + out [+ residual]) / BW), whole network = sum over layers.  Canonical bytes per
stored nonzero are sizeof(value) + 2 (16-bit offset) plus 4 * (c_out + 1) row pointers
per layer, whatever the packer really stores; layers kept dense count numel * sizeof.
"""
import json
import os

SM_COUNT = 148
FP32_LANES_PER_SM = 128
SM_MAX_MHZ = 1965.0
HBM_NOMINAL_GBS = 8000.0
HBM_FALLBACK_GBS = 6650.0

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def alu_peak_tflops(sm_mhz=SM_MAX_MHZ):
    """Plain-ALU peak: SMs x FP32 lanes x 2 flop x clock (an fp32 FMA or an int32 IMAD per lane per clock)."""
    return SM_COUNT * FP32_LANES_PER_SM * 2 * sm_mhz * 1e6 / 1e12


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured",
                "sm_max_mhz": float(d.get("sm_max_mhz", SM_MAX_MHZ))}
    return {"hbm_gbs": HBM_FALLBACK_GBS, "source": "fallback", "sm_max_mhz": SM_MAX_MHZ}


def layer_work(op, batch, dtype):
    """Algorithmic flops and bytes of one op at the given batch."""
    esz = 1 if dtype == "s8" else 4
    ho, wo = op.out_hw
    hi, wi = op.in_hw
    if op.kind in ("conv", "fc"):
        pixels = batch * ho * wo
        nnz = op.nnz
        flops = 2.0 * nnz * pixels
        if op.mask is None:
            wbytes = op.w.size * esz
        else:
            wbytes = nnz * (esz + 2) + 4 * (op.c_out + 1)
        in_b = batch * hi * wi * op.c_in * esz if op.kind == "conv" else batch * op.c_in * esz
        osz = {"f32": 4, "s8": 1, "s32": 4}[op.out]
        out_b = pixels * op.c_out * osz
        res_b = out_b if op.res >= 0 else 0
        return {"flops": flops, "wbytes": wbytes, "abytes": in_b + out_b + res_b, "nnz": nnz, "pixels": pixels}
    in_b = batch * hi * wi * op.c_in * esz
    out_b = batch * ho * wo * op.c_out * (4 if op.kind == "gavgpool" else esz)
    return {"flops": 0.0, "wbytes": 0, "abytes": in_b + out_b, "nnz": 0, "pixels": batch * ho * wo}


def layer_roof_us(work, r_tflops, bw_gbs):
    t_alu = work["flops"] / (r_tflops * 1e12)
    t_mem = (work["wbytes"] + work["abytes"]) / (bw_gbs * 1e9)
    return max(t_alu, t_mem) * 1e6, t_alu * 1e6, t_mem * 1e6


def family(op):
    """Kernel family an op runs in (mirrors the packer's dispatch)."""
    if op.kind == "conv":
        if op.groups > 1:
            return "dwconv"
        return "sconv_1x1" if (op.w.shape[1] * op.w.shape[2] == 1) else "sconv_kxk"
    if op.kind == "fc":
        return "sfc"
    return op.kind


def network_roofline(model, batch, r_tflops, bw_gbs):
    rows = []
    for op in model.ops:
        wk = layer_work(op, batch, model.dtype)
        t, ta, tm = layer_roof_us(wk, r_tflops, bw_gbs)
        rows.append({"name": op.name, "family": family(op), "t_roof_us": t, "t_alu_us": ta, "t_mem_us": tm, **wk})
    return rows
