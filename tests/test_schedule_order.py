"""Host logic of the two-stream schedule: the order in which a layer's inputs are taken."""
from paper_2311_01305_b200 import calibrate, synth


def test_schedule_order_is_a_permutation_with_the_lightest_weights_last():
    for wl in synth.workloads().values():
        fed = [i.name for i in wl.inputs if any(l.input == i.name for l in wl.linears)]
        order = calibrate.schedule_order(wl)
        assert sorted(order) == sorted(fed)
        if len(fed) >= 3:
            wbytes = {n: sum(l.c_out * l.c_in for l in wl.linears if l.input == n) for n in fed}
            assert wbytes[order[-1]] == min(wbytes.values())
            heavy = max(order[:-1], key=lambda n: wbytes[n])
            xbytes = {i.name: i.n_tokens * i.c_in for i in wl.inputs}
            after = order[order.index(heavy) + 1]
            assert after == order[-1] or xbytes[after] == max(xbytes[n] for n in order[:-1]) or \
                heavy == max(order[:-1], key=lambda n: xbytes[n])


def test_schedule_order_of_the_decoder_layers():
    wls = synth.workloads()
    assert calibrate.schedule_order(wls["llama7b_layer_w4w3_g128"]) == ["attn_in", "mlp_in", "down_in", "o_in"]
    assert calibrate.schedule_order(wls["opt125m_model_w8a8"]) == ["attn_in", "fc1_in", "fc2_in", "o_in"]
    assert calibrate.schedule_order(wls["opt66b_ffn_w8a8"]) == ["fc1_in", "fc2_in"]
