"""GPU parity of one denoising step of the latent-diffusion UNet (every linear and convolution but the first and last
is a Hadamard-quantized layer, with the network's own arithmetic between them) against the CPU oracle.

A reduced network with the topology of the benchmark's (four levels, two residual blocks per level, attention at three
resolutions, skip connections, step + class embedding) runs once on the device with every library call recorded.
(1) Layer by layer: each call's output is checked against the oracle applied to THE DEVICE'S OWN INPUT of that call, at
the tolerances of the single-layer tests (codes by the tie rule, outputs of quantized layers against the oracle's
rescale of the integer product of the device's codes, bf16 glue to one rounding).  (2) End to end: the predicted noise
against the oracle's forward in fp64 with the same parameters and static scales, as a relative rms distance."""
import numpy as np
import pytest

from paper_2512_05746_b200 import inputs
from hq_testutil import (PARITY_STATS, SCALE_RTOL, Y_BF16_RTOL, Y_F32_RTOL, attention_bound, check_codes, rel_err,
                         weight_integers)

pytestmark = pytest.mark.gpu

CFG = dict(batch=2, latent=32, base=128, attn_resolutions=(16, 8, 4), had_block=128, classes=10)
# Relative rms distance of the W4A8 prediction to the all-oracle forward: measured 4.3e-2 (codes on rounding ties and
# bf16 rounding boundaries, carried through 130 layers); a mis-wired network gives 0.5 or more.
E2E_RMS_BOUND_A8 = 8e-2


@pytest.fixture(scope="module")
def run():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2512_05746_b200 import binding as hq
    from paper_2512_05746_b200.unet import UNet
    cfg = inputs.unet_config(**CFG)
    P = inputs.unet_params(cfg, seed=0)
    I = inputs.unet_inputs(cfg, seed=0)
    net = UNet(cfg, P, hq, torch.device("cuda", 0)).build(cfg["batch"])
    x, t, y = torch.from_numpy(I["x"]), torch.from_numpy(I["t"]), torch.from_numpy(I["y"])
    net.calibrate(x, t, y)
    rec = []
    eps = net.forward(x, t, y, record=rec)
    torch.cuda.synchronize()
    hq.hq_check_status(net.status)
    return dict(torch=torch, hq=hq, cfg=cfg, P=P, I=I, net=net, rec=rec, eps=eps.cpu().numpy())


def host(tensor):
    return tensor.float().cpu().numpy().astype(np.float64)


def codes_of(r, rows, cols):
    return r["codes"].cpu().numpy()[:rows, :cols].view(np.int8)


def test_every_layer_matches_the_oracle_on_the_devices_own_input(run, oracle):
    hq, cfg, P, net = run["hq"], run["cfg"], run["P"], run["net"]
    G, heads = cfg["groups"], cfg["heads"]
    by_name = {r["name"]: r for r in run["rec"]}
    checked = {"q": 0, "g": 0}
    for r in run["rec"]:
        name, op = r["name"], r["op"]
        if op in ("conv3", "conv1"):
            x = host(r["x"])
            if r.get("x2") is not None:                            # a skip connection joined by concatenation, read in place
                x = np.concatenate([x, host(r["x2"])], axis=-1)
            Nb, H, W, C = x.shape
            w, b = P[name + ".w"], P[name + ".b"]
            stride = r.get("stride", 1)
            if r.get("pre_bias") is not None:                      # the step embedding, added in front of the normalisation
                x = x + host(r["pre_bias"])[:, None, None, :]
            xin = oracle.groupnorm(x, G, P[r["norm"] + ".gamma"], P[r["norm"] + ".beta"], net.EPS, "silu") if r.get("norm") else x
            pw = net.pw[name]
            static = float(r["static"].cpu()[0]) if op == "conv3" else None
            ref = oracle.qconv(xin, w, b, a_bits=4, w_bits=4, had_block=pw.desc.had_block, stride=stride, pad=w.shape[1] // 2,
                               weight_mode="folded", static_scale=static)
            q_gpu = codes_of(r, Nb * H * W, C)
            v = ref["v"].reshape(-1, C)
            if static is not None:
                v = np.clip(v, oracle.qmin(4) - 0.25, oracle.qmax(4) + 0.25)
            else:
                s_gpu = r["scales"].cpu().numpy()[: Nb * H * W]
                assert np.allclose(s_gpu, ref["s_a"], rtol=SCALE_RTOL, atol=0), name
            check_codes(q_gpu, ref["q"].reshape(-1, C), v, f"unet {name}")
            B = weight_integers(oracle, pw, w, 4, pw.desc.had_block, "folded").reshape(w.shape)
            qg = q_gpu.reshape(Nb, H, W, C)
            if static is not None:
                y_own = oracle.dequant(oracle.conv2d_int(qg, B, stride, 1), np.array([static], np.float32), pw.s_w, b, pw.alpha)
            else:
                y_own = oracle.conv2d_dequant_perpixel(qg, s_gpu, B, 1, 0, pw.s_w, b, pw.alpha)
            assert rel_err(host(r["y"]), y_own) <= Y_BF16_RTOL, name
            checked["q"] += 1
        elif op == "linear":
            x = host(r["x"])
            M, K = x.shape
            w, b = P[name + ".w"], P[name + ".b"]
            pw = net.pw[name]
            if r.get("norm"):
                Nb = r["Nb"]
                xin = oracle.groupnorm(x.reshape(Nb, M // Nb, 1, K), G, P[r["norm"] + ".gamma"], P[r["norm"] + ".beta"], net.EPS,
                                       "none").reshape(M, K)
            else:
                xin = x
            ref = oracle.qlinear(xin, w, b, a_bits=4, w_bits=4, had_block=pw.desc.had_block, weight_mode="folded")
            q_gpu, s_gpu = codes_of(r, M, K), r["scales"].cpu().numpy()[:M]
            assert np.allclose(s_gpu, ref["s_a"], rtol=SCALE_RTOL, atol=0), name
            check_codes(q_gpu, ref["q"], ref["v"], f"unet {name}")
            B = weight_integers(oracle, pw, w, 4, pw.desc.had_block, "folded")
            y_own = oracle.dequant(oracle.gemm_int(q_gpu, B), s_gpu, pw.s_w, b, pw.alpha)
            assert rel_err(host(r["y"]), y_own) <= Y_BF16_RTOL, name
            checked["q"] += 1
        else:
            out = host(r["out"])
            if op == "timestep_embedding":
                want = oracle.timestep_embedding(r["t"].cpu().numpy().astype(np.float64), cfg["base"])
                assert np.abs(out - want).max() <= 2.0 ** -8 + 2e-4, name
            elif op == "silu":
                assert rel_err(out, oracle.silu(host(r["x"]))) <= Y_BF16_RTOL, name
            elif op == "class_embed_add":
                before = host(by_name["time_embed.2"]["y"])
                table = host(net.bf["label_emb"])
                assert rel_err(out, before + table[r["labels"].cpu().numpy()]) <= Y_BF16_RTOL, name
            elif op == "add":
                assert rel_err(out, (host(r["a"]) + host(r["b"])).reshape(out.shape)) <= Y_BF16_RTOL, name
            elif op == "concat":
                assert np.array_equal(out, np.concatenate([host(r["a"]), host(r["b"])], axis=-1)), name
            elif op == "upsample":
                assert np.array_equal(out, oracle.upsample_nearest2x(host(r["x"]))), name
            elif op == "groupnorm_silu":
                want = oracle.groupnorm(host(r["x"]), G, P["out_norm.gamma"], P["out_norm.beta"], net.EPS, "silu")
                assert rel_err(out, want) <= Y_BF16_RTOL, name
            elif op == "conv_float":
                want = oracle.conv2d_float(host(r["x"]), P[name + ".w"], P[name + ".b"], 1, 1)
                assert rel_err(out, want) <= (Y_F32_RTOL if name == "out_conv" else Y_BF16_RTOL), name
            elif op == "attention":
                qkv = host(r["qkv"])
                Nb = r["Nb"]
                L, C = qkv.shape[0] // Nb, qkv.shape[1] // 3
                want = oracle.attention(qkv.reshape(Nb, L, 3 * C), heads).reshape(Nb * L, C)
                assert np.all(np.abs(out - want) <= attention_bound(oracle, qkv, Nb, L, C, heads, want)), name
            else:
                raise AssertionError(f"no check for {op}")
            checked["g"] += 1
    # every call of the forward was checked: 16 residual blocks x 3-4 layers, 11 attention blocks x 2, 6 resampling convs, 2 embedding linears
    assert checked["q"] == len([1 for tag, _, _ in net.tape if tag == "q"]) and checked["q"] >= 80
    assert checked["g"] == len([1 for tag, _, _ in net.tape if tag == "g"])
    # every residual block of the up-sampling path read [h | skip] in place, in its first and in its 1x1 skip convolution
    assert sum(1 for r in run["rec"] if r.get("x2") is not None) == 2 * sum(1 for r in run["rec"] if r["name"].startswith("up") and r["name"].endswith(".conv2"))
    # every residual block's second convolution took the block's embedding as its addend
    assert [r["name"] for r in run["rec"] if r.get("pre_bias") is not None] == [r["name"] for r in run["rec"] if r["name"].endswith(".conv2")]


def oracle_forward(run, oracle, a_bits, x=None):
    from oracle import unet_oracle
    cfg, P, I, net, torch = run["cfg"], run["P"], run["I"], run["net"], run["torch"]
    static = {k: float(v.cpu()[0]) for k, v in net.static.items()}
    Pd = dict(P)
    Pd["label_emb"] = net.bf["label_emb"].float().cpu().numpy()               # the table as the device holds it (bf16)
    if x is None:
        x = torch.from_numpy(I["x"]).to(torch.bfloat16).float().numpy()       # the latent as the device reads it
    return unet_oracle.forward(cfg, Pd, x, I["t"], I["y"], static, a_bits=a_bits, store=oracle.round_bf16)


def rms_rel(got, want):
    return float(np.sqrt(((got.astype(np.float64) - want) ** 2).mean() / (want ** 2).mean()))


def test_predicted_noise_with_8_bit_activations_close_to_the_all_oracle_forward(run, oracle):
    """End to end at W4A8, where a code that falls on the other side of a rounding tie is 1/16 of a 4-bit step: the
    predicted noise against the oracle's forward, which keeps every tensor between two operations in bf16 as the device
    does (the layers are defined with bf16 outputs).  A wrong skip connection, concatenation order, embedding or
    resampling anywhere in the sequence of calls gives a distance of order one."""
    torch, hq, cfg, P, I = run["torch"], run["hq"], run["cfg"], run["P"], run["I"]
    from paper_2512_05746_b200.unet import UNet
    net8 = UNet(cfg, P, hq, torch.device("cuda", 0), a_bits=8).build(cfg["batch"])
    x, t, y = torch.from_numpy(I["x"]), torch.from_numpy(I["t"]), torch.from_numpy(I["y"])
    net8.calibrate(x, t, y)
    got = net8.forward(x, t, y).cpu().numpy()
    hq.hq_check_status(net8.status)
    want = oracle_forward(dict(run, net=net8), oracle, 8)
    assert got.shape == want.shape and np.isfinite(got).all()
    rms = rms_rel(got, want)
    PARITY_STATS.append(dict(what="unet end to end W4A8 (batch 2, 32x32 latent, base 128)", rms_rel=rms))
    assert rms <= E2E_RMS_BOUND_A8, f"relative rms distance {rms:.3e}"
    assert 0.1 < np.sqrt((want ** 2).mean()) < 10.0            # not degenerate: the prediction has the scale of its input


def test_predicted_noise_with_4_bit_activations_within_the_networks_own_sensitivity(run, oracle):
    """End to end at W4A4.  The quantizer of Eq. 3 is discontinuous: a perturbation of relative size d in front of it
    moves a fraction of about d * sigma / step of the codes by a whole step, i.e. comes out as about sqrt(d); a chain of
    such layers carries ANY difference, however small, to a distance of order (step / sigma)^2 within a few layers.
    The device and the oracle agree on every layer given the same input (the test above) but differ in a few codes that
    sit on rounding ties, so their end-to-end distance is that level and no smaller.  The reference for it is the
    oracle against itself: the same forward with five of the latent's 6144 values moved by one bf16 step."""
    cfg, I, torch = run["cfg"], run["I"], run["torch"]
    want = oracle_forward(run, oracle, 4)
    got = run["eps"]
    assert got.shape == want.shape and np.isfinite(got).all()
    x = torch.from_numpy(I["x"]).to(torch.bfloat16).float().numpy()
    xp = x.copy()
    flat = xp.reshape(-1)
    for i in (11, 1500, 3001, 4444, 6000):
        flat[i] = flat[i] * (1.0 + 2.0 ** -7)                  # the neighbouring bf16 number
    own = rms_rel(oracle_forward(run, oracle, 4, x=xp), want)
    rms = rms_rel(got, want)
    PARITY_STATS.append(dict(what="unet end to end W4A4 (batch 2, 32x32 latent, base 128)", rms_rel=rms,
                             oracle_self_sensitivity=own))
    assert rms <= 1.25 * own + 0.02, f"device vs oracle {rms:.3f}, oracle vs minimally perturbed oracle {own:.3f}"
    # and the recorded block outputs agree exactly (to bf16) until the first code on a tie: the first residual block
    first = next(r for r in run["rec"] if r["name"] == "down0.res0.residual")
    trace = {}
    from oracle import unet_oracle
    Pd = dict(run["P"])
    Pd["label_emb"] = run["net"].bf["label_emb"].float().cpu().numpy()
    static = {k: float(v.cpu()[0]) for k, v in run["net"].static.items()}
    unet_oracle.forward(cfg, Pd, x, I["t"], I["y"], static, trace=trace, store=oracle.round_bf16)
    assert rms_rel(host(first["out"]), trace["down0.res0"]) <= 1e-3


def test_prediction_depends_on_step_and_class_of_its_own_sample_only(run):
    torch, I, net = run["torch"], run["I"], run["net"]
    t2 = I["t"].copy()
    t2[0] = (t2[0] + 500.0) % 1000.0
    other = net.forward(torch.from_numpy(I["x"]), torch.from_numpy(t2), torch.from_numpy(I["y"])).cpu().numpy()
    assert np.abs(other[0] - run["eps"][0]).max() > 0.05 and np.abs(other[1] - run["eps"][1]).max() < 1e-3
