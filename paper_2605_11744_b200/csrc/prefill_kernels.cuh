#pragma once
#include "mask.cuh"
