"""Cost model of App. D (bit operations) -- reporting only, TEST INFRASTRUCTURE like the rest of ``oracle``.

MAC(conv) = Cin*Cout*Nw*Nh*Kw*Kh/(Sw*Sh); BOPs = MAC*b_w*b_a; one Haar level on a C-channel W x H map costs
4*C*W*H*b_a, and level l works on a map 4^(l-1) times smaller; the inverse costs the same with Cout.
"""


def conv_mac(cin, cout, nw, nh, kw=1, kh=1, sw=1, sh=1):
    return cin * cout * nw * nh * kw * kh / (sw * sh)


def conv_bops(cin, cout, nw, nh, bits_w, bits_a, **kw):
    return conv_mac(cin, cout, nw, nh, **kw) * bits_w * bits_a


def haar_bops(channels, nw, nh, levels, bits_a):
    return sum(4 * channels * nw * nh * bits_a / 4 ** (l - 1) for l in range(1, levels + 1))


def wcc_bops(cin, cout, nw, nh, levels, gamma, bits_w, bits_a):
    """Compressed 1x1 conv on gamma*Nw*Nh columns plus the forward and inverse transforms."""
    return (gamma * conv_bops(cin, cout, nw, nh, bits_w, bits_a)
            + haar_bops(cin, nw, nh, levels, bits_a) + haar_bops(cout, nw, nh, levels, bits_a))
